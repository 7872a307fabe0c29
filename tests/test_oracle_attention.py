"""Pins for the attention oracle: none of them re-derives the oracle from itself."""
import math

import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo


def _case(seed, t_q, t_k, h_q, h_kv, d):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((t_q, h_q, d))
    k = rng.standard_normal((t_k, h_kv, d))
    v = rng.standard_normal((t_k, h_kv, d))
    return q, k, v


@pytest.mark.parametrize("t_q,t_k,h_q,h_kv", [(37, 37, 4, 4), (20, 20, 8, 2), (9, 30, 4, 2), (1, 17, 2, 1)])
@pytest.mark.parametrize("causal", [True, False])
def test_all_ones_mask_is_library_attention(t_q, t_k, h_q, h_kv, causal):
    """With every group active the result is ordinary (grouped-query) attention."""
    d = 16
    q, k, v = _case(1, t_q, t_k, h_q, h_kv, d)
    mask = np.ones((t_q, h_q // 2), dtype=bool)
    got = wo.masked_attention(q, k, v, mask, 2, causal=causal)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, k, v))   # [1, H, T, d]
    rep = h_q // h_kv
    tk, tv = tk.repeat_interleave(rep, dim=1), tv.repeat_interleave(rep, dim=1)
    allow = None
    if causal:   # bottom-right aligned causal mask: key j visible to query t iff j <= t + (T_k - T_q)
        allow = torch.arange(t_k)[None, :] <= (torch.arange(t_q)[:, None] + (t_k - t_q))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=allow)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-12)


def test_inactive_pairs_are_zero_and_active_pairs_unchanged():
    q, k, v = _case(2, 25, 25, 6, 3, 8)
    rng = np.random.default_rng(3)
    mask = rng.random((25, 3)) < 0.5
    full = wo.masked_attention(q, k, v, np.ones_like(mask), 2)
    got = wo.masked_attention(q, k, v, mask, 2)
    head_mask = np.repeat(mask, 2, axis=1)                       # [T, H_q]
    assert (got[~head_mask] == 0.0).all()
    np.testing.assert_array_equal(got[head_mask], full[head_mask])


def test_single_key_constant_v_and_first_row():
    q, k, v = _case(4, 6, 1, 2, 2, 4)
    got = wo.masked_attention(q, k, v, np.ones((6, 2), dtype=bool), 1)   # T_k = 1: delta = -5
    # only the last query sees the single key under the causal rule; non-causal everyone does
    got_nc = wo.masked_attention(q, k, v, np.ones((6, 2), dtype=bool), 1, causal=False)
    np.testing.assert_allclose(got_nc, np.broadcast_to(v[0], (6, 2, 4)), atol=1e-15)
    np.testing.assert_allclose(got[5], v[0], atol=1e-15)
    assert (got[:5] == 0.0).all()
    q, k, v = _case(5, 7, 7, 2, 1, 4)
    v[:] = np.array([1.0, -2.0, 3.0, 0.5])                       # same value vector at every key
    got = wo.masked_attention(q, k, v, np.ones((7, 1), dtype=bool), 2)
    np.testing.assert_allclose(got, np.broadcast_to(v[0, 0], (7, 2, 4)), atol=1e-14)
    q, k, v = _case(6, 7, 7, 2, 2, 4)
    got = wo.masked_attention(q, k, v, np.ones((7, 2), dtype=bool), 1)
    np.testing.assert_allclose(got[0], v[0], atol=1e-15)        # the first token sees only itself


def test_zero_query_averages_the_visible_keys():
    q, k, v = _case(7, 5, 8, 2, 1, 4)
    q[:] = 0.0
    got = wo.masked_attention(q, k, v, np.ones((5, 1), dtype=bool), 2)
    for t in range(5):
        np.testing.assert_allclose(got[t, 0], v[: t + 4, 0].mean(axis=0), atol=1e-14)   # delta = 3
        np.testing.assert_allclose(got[t, 1], v[: t + 4, 0].mean(axis=0), atol=1e-14)


def test_explicit_loops_on_a_tiny_case():
    t_q, t_k, h_q, h_kv, d, hpg = 4, 6, 4, 2, 3, 2
    q, k, v = _case(8, t_q, t_k, h_q, h_kv, d)
    mask = np.array([[1, 0], [0, 1], [1, 1], [0, 0]], dtype=bool)
    got = wo.masked_attention(q, k, v, mask, hpg, scale=0.7)
    for t in range(t_q):
        for h in range(h_q):
            want = [0.0] * d
            if mask[t, h // hpg]:
                hk = h // (h_q // h_kv)
                logits = [0.7 * sum(q[t, h, i] * k[j, hk, i] for i in range(d)) for j in range(t + (t_k - t_q) + 1)]
                z = sum(math.exp(l) for l in logits)
                for j, l in enumerate(logits):
                    for i in range(d):
                        want[i] += math.exp(l) / z * v[j, hk, i]
            np.testing.assert_allclose(got[t, h], want, rtol=1e-12, atol=1e-14)


def test_shifting_every_key_changes_nothing():
    """q.(k_j + c) = q.k_j + q.c adds the same number to every logit of a row."""
    q, k, v = _case(9, 11, 11, 2, 2, 8)
    mask = np.ones((11, 1), dtype=bool)
    a = wo.masked_attention(q, k, v, mask, 2)
    b = wo.masked_attention(q, k + np.linspace(-1, 1, 8), v, mask, 2)
    np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-12)


# ----------------------------------------------------------------------------- routed Q projection
def test_qproj_is_a_masked_library_matmul_and_matches_loops():
    rng = np.random.default_rng(12)
    T, D, G, NG = 9, 5, 4, 3
    x, w = rng.standard_normal((T, D)), rng.standard_normal((NG * G, D))
    mask = rng.random((T, NG)) < 0.5
    got = wo.qproj(x, w, mask, G)
    ref = (torch.from_numpy(x) @ torch.from_numpy(w).T).numpy()
    for t in range(T):
        for c in range(NG * G):
            want = sum(x[t, i] * w[c, i] for i in range(D)) if mask[t, c // G] else 0.0
            assert abs(got[t, c] - want) < 1e-12
            if mask[t, c // G]:
                assert abs(got[t, c] - ref[t, c]) < 1e-12
    assert (wo.qproj(x, w, np.zeros_like(mask), G) == 0).all()
    np.testing.assert_allclose(wo.qproj(x, w, np.ones_like(mask), G), ref, atol=1e-12)
