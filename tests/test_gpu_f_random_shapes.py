"""Seeded random shapes through every tensor-core path: ragged token counts, odd group counts,
variable per-token budgets, empty and full groups.  Each case is checked against the oracle."""
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


def _mask(rng, T, NG):
    """Bernoulli mask with a random density; now and then a group nobody or everybody selects."""
    m = rng.random((T, NG)) < rng.uniform(0.1, 0.9)
    if NG > 2 and rng.random() < 0.5:
        m[:, rng.integers(0, NG)] = False
    if NG > 2 and rng.random() < 0.5:
        m[:, rng.integers(0, NG)] = True
    return m


@pytest.mark.parametrize("seed", range(8))
def test_ffn_random_shapes(ctx, seed):
    from paper_2607_28418_b200 import binding
    rng = np.random.default_rng(1000 + seed)
    G = int(rng.choice([64, 128, 256]))
    NG = int(rng.integers(2, 11))
    D = 64 * int(rng.integers(2, 9))
    T = int(rng.choice([int(rng.integers(1, 65)), int(rng.integers(65, 900))]))
    cfg = synth.WideConfig("rnd", tokens=T, hidden=D, d_ff=NG * G, group=G, k=1)
    case = synth.make_ffn_case(cfg, seed)
    mask = _mask(rng, T, NG)
    dev = {k: to_dev(case[k], "bf16") for k in ("x", "w_gate", "w_up", "w_down")}
    meta = meta_to_dev(wo.reorder(mask, 128)) if T > 64 else None
    y = binding.wide_ffn(ctx, dev["x"], dev["w_gate"], dev["w_up"], dev["w_down"], G, bits_to_dev(wo.pack_mask_bits(mask)), meta)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    ref = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, G)
    assert_close(y, ref, f"ffn T={T} D={D} NG={NG} G={G}")


@pytest.mark.parametrize("seed", range(6))
def test_oproj_qproj_random_shapes(ctx, seed):
    from paper_2607_28418_b200 import binding
    rng = np.random.default_rng(2000 + seed)
    G = int(rng.choice([128, 256, 512]))
    NG = int(rng.integers(1, 9))
    D = 64 * int(rng.integers(2, 9))
    T = int(rng.choice([int(rng.integers(1, 65)), int(rng.integers(65, 700))]))
    K = NG * G
    mask = _mask(rng, T, NG)
    bits = bits_to_dev(wo.pack_mask_bits(mask))
    meta = meta_to_dev(wo.reorder(mask, 128))
    a = synth.make_activations(rng, T, K, "bf16", "random")
    w_o = synth.make_weight(rng, D, K, 0.02, "bf16")
    y = binding.wide_oproj(ctx, to_dev(a, "bf16"), to_dev(w_o, "bf16"), G, bits, meta if T > 64 else None)
    assert_close(y, wo.oproj(a, w_o, mask, G), f"oproj T={T} D={D} NG={NG} G={G}")
    x = synth.make_activations(rng, T, D, "bf16", "random")
    w_q = synth.make_weight(rng, K, D, 0.02, "bf16")
    yq = binding.wide_qproj(ctx, to_dev(x, "bf16"), to_dev(w_q, "bf16"), G, meta)
    ref = wo.qproj(x, w_q, mask, G)
    assert (yq.float().cpu().numpy()[~wo.expand_group_mask(mask, G)] == 0.0).all()
    assert_close(yq, ref, f"qproj T={T} D={D} NG={NG} G={G}")
    torch.cuda.synchronize()
    assert ctx.status() == 0


@pytest.mark.parametrize("seed", range(6))
def test_attn_random_shapes(ctx, seed):
    from paper_2607_28418_b200 import binding
    rng = np.random.default_rng(3000 + seed)
    hd = int(rng.choice([64, 128]))
    h_kv = int(rng.choice([1, 2, 4]))
    rep = int(rng.choice([1, 2, 4]))
    h_q = h_kv * rep
    hpg = int(rng.choice([d for d in (1, 2, 4, 8) if h_q % d == 0]))
    t_q = int(rng.integers(1, 700))
    t_k = t_q + int(rng.choice([0, 0, int(rng.integers(1, 300))]))
    causal = bool(rng.random() < 0.7)
    case = synth.make_attn_case(seed, t_q, t_k, h_q, h_kv, hd)
    mask = _mask(rng, t_q, h_q // hpg)
    meta = meta_to_dev(wo.reorder(mask, 128))
    o = binding.wide_attn(ctx, to_dev(case["q"].reshape(t_q, -1), "bf16"), to_dev(case["k"].reshape(t_k, -1), "bf16"),
                          to_dev(case["v"].reshape(t_k, -1), "bf16"), h_q, h_kv, hpg, meta, causal=causal)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    ref = wo.masked_attention(case["q"], case["k"], case["v"], mask, hpg, causal=causal)
    assert_close(o.reshape(t_q, h_q, hd), ref, f"attn Tq={t_q} Tk={t_k} Hq={h_q} Hkv={h_kv} d={hd} hpg={hpg} causal={causal}")
