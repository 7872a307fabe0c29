"""Pins for the oracle's routing, top-k, bit packing and mask reordering.

None of these re-types the oracle's own formula: they use exact rational brute force,
closed-form routers, a hand-worked fixture, and the invariants the paper states for the
sorted layout (Section 3.3 and Appendix B).
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_fixture(path):
    sections, name = {}, None
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line[0].isalpha():
                name = line
                sections[name] = []
            else:
                sections[name].append([int(v) for v in line.split()])
    return sections


# ----------------------------------------------------------------------------- scores / top-k
def test_scores_match_exact_rational_brute_force():
    rng = np.random.default_rng(0)
    T, D, NG = 5, 12, 7
    x = synth.round_to_bf16(rng.standard_normal((T, D)).astype(np.float32))
    w = synth.round_to_bf16(rng.standard_normal((NG, D)).astype(np.float32))
    s = wo.route_scores(x, w)
    for t in range(T):
        for g in range(NG):
            exact = sum(Fraction(float(x[t, i])) * Fraction(float(w[g, i])) for i in range(D))
            assert abs(Fraction(float(s[t, g])) - exact) <= abs(exact) * Fraction(1, 10**14) + Fraction(1, 10**300)


def test_scores_not_transposed():
    # x = e_i picks column i of the router: s[t, g] = w[g, i]
    D, NG = 6, 4
    w = np.arange(NG * D, dtype=np.float32).reshape(NG, D)
    x = np.eye(D, dtype=np.float32)
    s = wo.route_scores(x, w)
    assert s.shape == (D, NG)
    for i in range(D):
        for g in range(NG):
            assert s[i, g] == w[g, i]


def test_topk_brute_force_rank_definition():
    # group g is selected iff fewer than k groups beat it under (score desc, index asc)
    rng = np.random.default_rng(1)
    T, NG = 40, 11
    s = rng.standard_normal((T, NG))
    s[3, :] = 0.0                       # full tie
    s[4, [2, 7, 9]] = 1.5               # partial ties at the top
    s[5, :] = np.round(s[5, :])         # many ties
    for k in (0, 1, 4, 10, 11):
        m = wo.mask_topk(s, k)
        for t in range(T):
            for g in range(NG):
                beats = sum(1 for h in range(NG)
                            if s[t, h] > s[t, g] or (s[t, h] == s[t, g] and h < g))
                assert m[t, g] == (beats < k)
        assert (m.sum(axis=1) == k).all()


def test_topk_ties_prefer_lower_index_and_extremes():
    s = np.zeros((2, 6))
    m = wo.mask_topk(s, 3)
    assert m.tolist() == [[True, True, True, False, False, False]] * 2
    assert not wo.mask_topk(s, 0).any()
    assert wo.mask_topk(s, 6).all()


def test_topk_per_token_budget():
    rng = np.random.default_rng(2)
    s = rng.standard_normal((9, 8))
    kt = np.array([0, 1, 2, 3, 4, 5, 6, 7, 8])
    m = wo.mask_topk(s, kt)
    assert (m.sum(axis=1) == kt).all()
    for t in range(9):
        if 0 < kt[t] < 8:
            assert s[t][m[t]].min() >= s[t][~m[t]].max()


def test_one_hot_router_closed_form():
    # router row g = e_g  =>  score[t, g] = x[t, g]  => mask marks the k largest coordinates
    rng = np.random.default_rng(3)
    T, NG, D = 16, 8, 8
    x = rng.permutation(T * D).reshape(T, D).astype(np.float32)  # all distinct
    w = np.eye(NG, D, dtype=np.float32)
    m = wo.mask_topk(wo.route_scores(x, w), 3)
    for t in range(T):
        top = set(np.argsort(-x[t])[:3].tolist())
        assert set(np.nonzero(m[t])[0].tolist()) == top


def test_pair_argmax_closed_cases():
    rng = np.random.default_rng(4)
    T, D, r, NG = 10, 16, 4, 6
    x = rng.standard_normal((T, D))
    w1 = rng.standard_normal((D, r))
    w2 = rng.standard_normal((r, 2 * NG))
    R = wo.route_logits_pair(x, w1, w2)
    assert R.shape == (T, NG, 2)
    m = wo.mask_pair_argmax(R)
    # equals the sign test of class-0 minus class-1 logit, computed by brute force
    for t in range(T):
        u = [sum(x[t, i] * w1[i, j] for i in range(D)) for j in range(r)]
        for g in range(NG):
            l0 = sum(u[j] * w2[j, 2 * g] for j in range(r))
            l1 = sum(u[j] * w2[j, 2 * g + 1] for j in range(r))
            if abs(l0 - l1) > 1e-9:
                assert m[t, g] == (l0 > l1)
    # class-1 logit pushed to -inf / +inf -> all execute / all skip; exact tie executes
    big = np.zeros((T, NG, 2))
    big[..., 1] = -np.inf
    assert wo.mask_pair_argmax(big).all()
    big[..., 1] = np.inf
    assert not wo.mask_pair_argmax(big).any()
    assert wo.mask_pair_argmax(np.zeros((T, NG, 2))).all()


def test_pack_unpack_bits():
    rng = np.random.default_rng(5)
    for NG in (1, 16, 31, 32, 33, 86, 224):
        m = rng.random((13, NG)) < 0.5
        bits = wo.pack_mask_bits(m)
        assert bits.shape == (13, (NG + 31) // 32) and bits.dtype == np.uint32
        for t in range(13):
            for g in range(NG):
                assert ((int(bits[t, g // 32]) >> (g % 32)) & 1) == int(m[t, g])
            # unused high bits stay zero
            total = sum(bin(int(wd)).count("1") for wd in bits[t])
            assert total == int(m[t].sum())
        assert (wo.unpack_mask_bits(bits, NG) == m).all()


# ----------------------------------------------------------------------------- reorder
def test_reorder_hand_worked_fixture():
    fx = _read_fixture(os.path.join(GOLDEN, "reorder_hand_worked.txt"))
    mask = np.array(fx["mask"], dtype=bool)
    r = wo.reorder(mask, tile_m=3)
    assert r["perm"].tolist() == fx["perm"]
    assert r["counts"].tolist() == fx["counts"][0]
    assert r["tile_map"].tolist() == fx["tile_map"]
    assert r["tile_any"].tolist() == fx["tile_any"]
    assert r["work_list"].tolist() == fx["work_list"]
    assert r["n_work"] == len(fx["work_list"])
    assert r["union_list"].tolist() == fx["union_list"][0]
    assert r["offsets"].tolist() == fx["offsets"][0]
    assert wo.pack_mask_bits(mask)[:, 0].tolist() == fx["mask_bits"][0]


@pytest.mark.parametrize("T,NG,tile_m,p", [(1, 1, 16, 0.5), (50, 5, 16, 0.5), (130, 33, 32, 0.3),
                                           (257, 16, 128, 0.9), (64, 7, 128, 0.0), (64, 7, 16, 1.0)])
def test_reorder_invariants(T, NG, tile_m, p):
    mask = synth.bernoulli_mask(T * 31 + NG, T, NG, p)
    r = wo.reorder(mask, tile_m)
    perm, sm, counts = r["perm"], r["sorted_mask"], r["counts"]
    n_tiles = (T + tile_m - 1) // tile_m
    for g in range(NG):
        assert sorted(perm[g].tolist()) == list(range(T))                    # a permutation
        assert (counts[g] == mask[:, g].sum())                               # column sums
        col = sm[:, g].astype(int)
        assert (np.diff(col) <= 0).all()                                     # monotone non-increasing
        assert (sm[:, g] == mask[perm[g], g]).all()                          # M~[j,g] = M[I[j,g],g]
        c = int(counts[g])
        assert (np.diff(perm[g, :c]) > 0).all() and (np.diff(perm[g, c:]) > 0).all()  # stable
        # level-0 predicate equals the first sorted entry of the tile (monotone shortcut)
        for m in range(n_tiles):
            assert r["tile_map"][m, g] == int(sm[m * tile_m, g])
            assert r["tile_map"][m, g] == int(m * tile_m < c)
        # at most one partially active tile per group
        partial = sum(1 for m in range(n_tiles)
                      if 0 < sm[m * tile_m:(m + 1) * tile_m, g].sum() < min(tile_m, T - m * tile_m))
        assert partial <= 1
    assert int(counts.sum()) == int(mask.sum())
    assert r["union_list"].tolist() == [g for g in range(NG) if mask[:, g].any()]
    assert r["n_work"] == int(sum((int(c) + tile_m - 1) // tile_m for c in counts))
    wl = r["work_list"].tolist()
    assert wl == sorted(wl, key=lambda mg: (mg[1], mg[0]))
    assert r["offsets"][0] == 0 and (np.diff(r["offsets"]) % tile_m == 0).all()
    assert (np.diff(r["offsets"]) >= counts).all()


def test_reorder_single_column_is_textbook_stable_partition():
    rng = np.random.default_rng(7)
    col = rng.random(200) < 0.4
    r = wo.reorder(col[:, None], 16)
    keys = np.where(col, 0, 1)
    assert r["perm"][0].tolist() == np.argsort(keys, kind="stable").tolist()


def test_union_single_token_is_its_own_groups():
    m = synth.random_mask(3, 1, 40, 13)
    r = wo.reorder(m, 128)
    assert r["union_list"].tolist() == np.nonzero(m[0])[0].tolist()
    assert r["n_union"] == 13


# ----------------------------------------------------------------------------- token clustering
def test_cluster_tokens_permutation_grouping_and_stability():
    rng = np.random.default_rng(12)
    T, NG = 300, 70
    protos = rng.random((5, NG)) < 0.5
    which = rng.integers(0, 5, size=T)
    mask = protos[which]
    c = wo.cluster_tokens(mask)
    order, rank = c["token_order"], c["token_rank"]
    assert sorted(order.tolist()) == list(range(T))
    assert (rank[order] == np.arange(T)).all() and (order[rank] == np.arange(T)).all()
    bits = wo.pack_mask_bits(mask)
    keys = np.array([wo.mask_key(bits[t], NG) for t in range(T)])
    assert ((0 <= keys) & (keys < 256)).all()
    assert (np.diff(keys[order]) >= 0).all()                        # sorted by key
    for p in range(T - 1):                                           # stable inside a key
        if keys[order[p]] == keys[order[p + 1]]:
            assert order[p] < order[p + 1]
    # identical masks are neighbours unless two prototypes collide on the 8-bit key
    proto_keys = {wo.mask_key(wo.pack_mask_bits(protos[i:i + 1])[0], NG) for i in range(5)}
    if len(proto_keys) == 5:
        runs = 1 + int((np.diff(which[order]) != 0).sum())
        assert runs == len(set(which.tolist()))


def test_mask_key_is_the_header_hash():
    # more than 32 groups: two worked values of h = (h ^ w) * 0x01000193 from h0 = 0x811C9DC5, top byte
    assert wo.mask_key([0, 0], 40) == ((((0x811C9DC5 * 0x01000193) & 0xFFFFFFFF) * 0x01000193) & 0xFFFFFFFF) >> 24
    h = ((0x811C9DC5 ^ 0xFFFFFFFF) * 0x01000193) & 0xFFFFFFFF
    h = ((h ^ 0x1) * 0x01000193) & 0xFFFFFFFF
    assert wo.mask_key([0xFFFFFFFF, 1], 33) == h >> 24
    # up to 32 groups: the decisions for groups 0..7 themselves
    assert wo.mask_key([0b1_0110_0101], 10) == 0b0110_0101
    assert wo.mask_key([0xFFFFFF00], 32) == 0


def test_cluster_tokens_few_groups_tiles_agree_on_leading_decisions():
    """With a handful of groups and a mask of its own per token, tiles of the clustered order still
    skip blocks: the sorted order is lexicographic in the decisions for groups 7..0, so 32 tiles of
    128 tokens agree on about five of them."""
    T, NG, k = 4096, 10, 5
    rng = np.random.default_rng(5)
    mask = wo.mask_topk(rng.standard_normal((T, NG)), k)
    order = wo.cluster_tokens(mask)["token_order"]
    def active_blocks(m):
        return sum(int(m[i:i + 128].any(axis=0).sum()) for i in range(0, T, 128))
    assert active_blocks(mask) == 32 * NG                     # token order: nothing to skip
    assert active_blocks(mask[order]) <= 0.87 * 32 * NG       # clustered order: about one block in six drops out
    keys = np.array([wo.mask_key(b, NG) for b in wo.pack_mask_bits(mask)])
    assert (np.diff(keys[order]) >= 0).all()


# ----------------------------------------------------------------------------- gather / scatter
def test_gather_then_unpermute_full_mask_is_identity():
    rng = np.random.default_rng(8)
    T, NG, G = 37, 5, 4
    dense = rng.standard_normal((T, NG * G)).astype(np.float32)
    r = wo.reorder(np.ones((T, NG), dtype=bool), 16)
    packed = wo.gather_packed(dense, r["perm"], r["counts"], r["offsets"], G)
    back = wo.unpermute(packed, r["perm"], r["counts"], r["offsets"], T, G)
    assert (back == dense).all()


def test_gather_then_unpermute_masks_groupwise():
    rng = np.random.default_rng(9)
    T, NG, G = 45, 6, 8
    dense = rng.standard_normal((T, NG * G)).astype(np.float32)
    mask = synth.bernoulli_mask(11, T, NG, 0.5)
    r = wo.reorder(mask, 16)
    packed = wo.gather_packed(dense, r["perm"], r["counts"], r["offsets"], G)
    assert packed.shape == (int(r["offsets"][-1]), G)
    back = wo.unpermute(packed, r["perm"], r["counts"], r["offsets"], T, G)
    for t in range(T):
        for g in range(NG):
            blk = back[t, g * G:(g + 1) * G]
            if mask[t, g]:
                assert (blk == dense[t, g * G:(g + 1) * G]).all()
            else:
                assert (blk == 0).all()


def test_packed_layout_matches_hand_worked_fixture():
    """gather_packed and unpermute each against a layout worked out by hand (Algorithm 2's scatter
    epilogue): a mistake both functions share, e.g. in the row order of the packed buffer, would
    survive the round-trip tests above but not this one."""
    fx = _read_fixture(os.path.join(GOLDEN, "packed_hand_worked.txt"))
    mask = np.array(fx["mask"], dtype=bool)
    r = wo.reorder(mask, 2)
    assert r["perm"].tolist() == fx["perm"]
    assert r["counts"].tolist() == fx["counts"][0]
    assert r["offsets"].tolist() == fx["offsets"][0]
    dense = np.array(fx["dense"], dtype=np.float32)
    packed = wo.gather_packed(dense, r["perm"], r["counts"], r["offsets"], 2)
    assert packed.tolist() == fx["packed"]
    back = wo.unpermute(np.array(fx["packed"], dtype=np.float32), np.array(fx["perm"], dtype=np.int32),
                        np.array(fx["counts"][0]), np.array(fx["offsets"][0]), 5, 2)
    assert back.tolist() == fx["scattered"]


# ----------------------------------------------------------------------------- pair router on the normalised input
def test_rmsnorm_matches_plain_loops():
    rng = np.random.default_rng(21)
    x = rng.standard_normal((5, 12)) * 3.0
    w = rng.standard_normal(12)
    got = wo.rmsnorm(x, w, 1e-5)
    for t in range(5):
        ms = sum(float(v) ** 2 for v in x[t]) / 12
        for i in range(12):
            assert abs(got[t, i] - x[t, i] / math.sqrt(ms + 1e-5) * w[i]) <= 1e-14 * (1 + abs(got[t, i]))
    # a row of unit mean square and no weight passes through (eps = 0)
    u = np.ones((1, 7))
    assert np.allclose(wo.rmsnorm(u, None, 0.0), u, rtol=0, atol=0)


def test_pair_router_on_normalised_input_by_loops_and_scale_invariance():
    rng = np.random.default_rng(22)
    T, D, r, NG = 6, 10, 3, 4
    x = rng.standard_normal((T, D))
    g = rng.standard_normal(D)
    w1 = rng.standard_normal((D, r))
    w2 = rng.standard_normal((r, 2 * NG))
    eps = 1e-6
    logits = wo.route_logits_pair_norm(x, g, eps, w1, w2)
    assert logits.shape == (T, NG, 2)
    for t in range(T):
        rms = math.sqrt(sum(float(v) ** 2 for v in x[t]) / D + eps)
        xh = [float(x[t, i]) / rms * float(g[i]) for i in range(D)]
        u = [sum(xh[i] * float(w1[i, c]) for i in range(D)) for c in range(r)]
        for n in range(2 * NG):
            ref = sum(u[c] * float(w2[c, n]) for c in range(r))
            assert abs(logits[t, n // 2, n % 2] - ref) <= 1e-12 * (1 + abs(ref))
    mask = wo.mask_pair_argmax(logits)
    # the decision ignores a positive scale of the row: the normalisation's 1/rms drops out, and so
    # does any rescaling of a token
    unscaled = wo.mask_pair_argmax(wo.route_logits_pair(x * g[None, :], w1, w2))
    assert (mask == unscaled).all()
    assert (wo.mask_pair_argmax(wo.route_logits_pair_norm(x * np.array([[0.01], [3.0], [1.0], [250.0], [7.0], [0.5]]),
                                                          g, 0.0, w1, w2)) == mask).all()
    # an all-zero token has all-zero logits: every pair ties, class 0 wins, everything executes
    z = wo.mask_pair_argmax(wo.route_logits_pair_norm(np.zeros((1, D)), g, eps, w1, w2))
    assert z.all()
