"""Pins for the oracle's masked FFN (Eq. 3) and masked O-projection (Eq. 2 / Eq. 10).

Closed cases: all-ones mask = dense SwiGLU (library routine), all-zero = 0, one active
group = brute-force sum over that group's channels, additivity over disjoint masks
(Eq. 10), the per-token gather formulations of Appendix A, constant-weight closed forms.
"""
import math

import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth


def _tiny(seed, T=6, D=8, NG=4, G=4):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, D))
    wg = rng.standard_normal((NG * G, D)) * 0.5
    wu = rng.standard_normal((NG * G, D)) * 0.5
    wd = rng.standard_normal((D, NG * G)) * 0.5
    return x, wg, wu, wd


def _brute_ffn_token(x_t, wg, wu, wd, groups, G):
    """Straight loops over the channels of the listed groups only."""
    D = len(x_t)
    y = [0.0] * wd.shape[0]
    for g in groups:
        for c in range(g * G, (g + 1) * G):
            a = sum(x_t[i] * wg[c, i] for i in range(D))
            b = sum(x_t[i] * wu[c, i] for i in range(D))
            h = a / (1.0 + math.exp(-a)) * b
            for n in range(wd.shape[0]):
                y[n] += h * wd[n, c]
    return y


def test_all_ones_equals_dense_swiglu_library():
    cfg = synth.CONFIGS["tiny"]
    case = synth.make_ffn_case(cfg, 0)
    mask = np.ones((cfg.tokens, cfg.n_groups), dtype=bool)
    y = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, cfg.group)
    x, wg, wu, wd = (torch.from_numpy(case[k]).double() for k in ("x", "w_gate", "w_up", "w_down"))
    ref = (torch.nn.functional.silu(x @ wg.T) * (x @ wu.T)) @ wd.T
    np.testing.assert_allclose(y, ref.numpy(), rtol=1e-11, atol=1e-13)


def test_all_zero_mask_gives_exact_zero():
    x, wg, wu, wd = _tiny(1)
    y = wo.ffn(x, wg, wu, wd, np.zeros((6, 4), dtype=bool), 4)
    assert (y == 0).all()
    a = np.random.default_rng(0).standard_normal((6, 16))
    assert (wo.oproj(a, wd, np.zeros((6, 4), dtype=bool), 4) == 0).all()


@pytest.mark.parametrize("g", [0, 1, 3])
def test_single_group_brute_force(g):
    x, wg, wu, wd = _tiny(2)
    mask = np.zeros((6, 4), dtype=bool)
    mask[:, g] = True
    mask[4, g] = False   # one token with nothing active
    y = wo.ffn(x, wg, wu, wd, mask, 4)
    for t in range(6):
        ref = _brute_ffn_token(x[t], wg, wu, wd, [g] if mask[t, g] else [], 4)
        np.testing.assert_allclose(y[t], ref, rtol=1e-12, atol=1e-14)


def test_arbitrary_mask_brute_force_and_token_independence():
    x, wg, wu, wd = _tiny(3, T=5, D=6, NG=5, G=3)
    mask = synth.bernoulli_mask(4, 5, 5, 0.5)
    y = wo.ffn(x, wg, wu, wd, mask, 3)
    for t in range(5):
        ref = _brute_ffn_token(x[t], wg, wu, wd, np.nonzero(mask[t])[0].tolist(), 3)
        np.testing.assert_allclose(y[t], ref, rtol=1e-12, atol=1e-14)
    # a row of the output depends only on its own token and mask row
    y_row = wo.ffn(x[2:3], wg, wu, wd, mask[2:3], 3)
    np.testing.assert_allclose(y_row[0], y[2], rtol=1e-13, atol=1e-15)


def test_additivity_over_disjoint_masks():
    x, wg, wu, wd = _tiny(5, T=9, D=8, NG=6, G=4)
    m = synth.bernoulli_mask(6, 9, 6, 0.6)
    m1 = m & (np.arange(6)[None, :] % 2 == 0)
    m2 = m & ~m1
    y = wo.ffn(x, wg, wu, wd, m, 4)
    np.testing.assert_allclose(y, wo.ffn(x, wg, wu, wd, m1, 4) + wo.ffn(x, wg, wu, wd, m2, 4),
                               rtol=1e-12, atol=1e-14)
    per_group = sum(wo.ffn(x, wg, wu, wd, m & (np.arange(6)[None, :] == g), 4) for g in range(6))
    np.testing.assert_allclose(y, per_group, rtol=1e-12, atol=1e-14)


def test_constant_weight_closed_form():
    # x = s * 1, Wg = a, Wu = b, Wd = w (constants): y[t, n] = k_t * G * silu(a s D) * (b s D) * w
    T, D, NG, G = 4, 5, 6, 3
    s, a, b, w = 0.3, -0.2, 0.7, 0.11
    x = np.full((T, D), s)
    mask = np.zeros((T, NG), dtype=bool)
    for t in range(T):
        mask[t, : t + 1] = True
    y = wo.ffn(x, np.full((NG * G, D), a), np.full((NG * G, D), b), np.full((D, NG * G), w), mask, G)
    pre = a * s * D
    h = pre / (1.0 + math.exp(-pre)) * (b * s * D)
    assert h < 0  # the sign of SiLU at a negative argument matters here
    for t in range(T):
        np.testing.assert_allclose(y[t], np.full(D, (t + 1) * G * h * w), rtol=1e-12)


def test_per_token_selected_group_sums_agree():
    """Appendix A states the pruned FFN per token: a token that selected R groups computes gate
    and up only for the R*G channels of those groups and reduces the down projection over the
    same channels.  Written here as plain loops over tokens, selected groups and channels."""
    x, wg, wu, wd = _tiny(7, T=7, D=6, NG=5, G=4)
    G = 4
    mask = synth.random_mask(8, 7, 5, 2)
    y_ref = np.zeros((7, wd.shape[0]))
    for t in range(7):
        for g in range(5):
            if not mask[t, g]:
                continue
            for c in range(g * G, (g + 1) * G):
                gate = sum(float(x[t, i]) * float(wg[c, i]) for i in range(6))
                up = sum(float(x[t, i]) * float(wu[c, i]) for i in range(6))
                h = gate / (1.0 + math.exp(-gate)) * up
                for n in range(wd.shape[0]):
                    y_ref[t, n] += h * float(wd[n, c])
    np.testing.assert_allclose(wo.ffn(x, wg, wu, wd, mask, G), y_ref, rtol=1e-12, atol=1e-14)


def test_topk_all_groups_is_dense():
    cfg = synth.CONFIGS["tiny"]
    case = synth.make_ffn_case(cfg, 1, tokens=16)
    out = wo.layer_ffn(case["x"], case["w_router"], case["w_gate"], case["w_up"], case["w_down"],
                       cfg.group, cfg.n_groups, 32)
    assert out["mask"].all()
    dense = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"],
                   np.ones((16, cfg.n_groups), dtype=bool), cfg.group)
    assert (out["y"] == dense).all()


# ----------------------------------------------------------------------------- O-projection
def test_oproj_equals_masked_library_matmul():
    rng = np.random.default_rng(10)
    T, NG, G, D = 12, 5, 8, 10
    a = rng.standard_normal((T, NG * G))
    w = rng.standard_normal((D, NG * G))
    mask = synth.bernoulli_mask(12, T, NG, 0.5)
    y = wo.oproj(a, w, mask, G)
    at = torch.from_numpy(a) * torch.from_numpy(mask).repeat_interleave(G, dim=1)
    np.testing.assert_allclose(y, (at @ torch.from_numpy(w).T).numpy(), rtol=1e-12, atol=1e-13)


def test_oproj_brute_force_group_sums():
    rng = np.random.default_rng(11)
    T, NG, G, D = 4, 3, 2, 3
    a = rng.standard_normal((T, NG * G))
    w = rng.standard_normal((D, NG * G))
    mask = np.array([[1, 0, 1], [0, 0, 0], [1, 1, 1], [0, 1, 0]], dtype=bool)
    y = wo.oproj(a, w, mask, G)
    for t in range(T):
        for n in range(D):
            ref = 0.0
            for g in range(NG):
                if mask[t, g]:
                    for c in range(g * G, (g + 1) * G):
                        ref += a[t, c] * w[n, c]
            assert abs(y[t, n] - ref) < 1e-13


def test_oproj_head_major_group_to_channel_map():
    # group g covers channels [g*G, (g+1)*G): a one-hot attention output on channel c only
    # reaches the output when group c // G is active.
    NG, G, D = 4, 3, 5
    w = np.arange(D * NG * G, dtype=np.float64).reshape(D, NG * G) + 1
    for c in range(NG * G):
        a = np.zeros((1, NG * G))
        a[0, c] = 1.0
        for g in range(NG):
            mask = np.zeros((1, NG), dtype=bool)
            mask[0, g] = True
            y = wo.oproj(a, w, mask, G)
            expect = w[:, c] if g == c // G else np.zeros(D)
            assert (y[0] == expect).all()


# ----------------------------------------------------------------------------- inputs
def test_synth_bf16_rounding_and_determinism():
    a = np.array([1.0, 1.00390625, 1.01171875, -3.1415927, 0.0], dtype=np.float32)
    r = synth.round_to_bf16(a)
    # 1.00390625 = 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7 -> even mantissa (1.0)
    # 1.01171875 = 1 + 3*2^-8 is a tie between 1 + 2^-7 and 1 + 2^-6 -> even mantissa (1 + 2^-6)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == np.float32(1.015625)
    assert (synth.from_bf16_bits(synth.to_bf16_bits(r)) == r).all()
    t = torch.from_numpy(a).to(torch.bfloat16).float().numpy()
    assert (r == t).all()
    c1 = synth.make_ffn_case(synth.CONFIGS["tiny"], 3)
    c2 = synth.make_ffn_case(synth.CONFIGS["tiny"], 3)
    assert all((c1[k] == c2[k]).all() for k in c1)
    cl = synth.make_ffn_case(synth.CONFIGS["tiny"].with_(router="clustered"), 3)
    assert len({row.tobytes() for row in cl["x"]}) <= 4
