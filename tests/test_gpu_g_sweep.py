"""GPU parity at every point of the sparsity sweep (8B-shaped FFN: hidden 4096, d_ff 14336).

Group size 64 / 128 / 256  x  active fraction 75 % / 50 % / 25 %  x  router random / clustered, at
4096 prefill tokens and at decode batch 16: the 36 points the benchmark's sweep table reports.  At
every point the mask and the reorder metadata are compared bit for bit and EVERY output row is
compared with the oracle (an output row depends only on its own token and mask row, Eq. 3).

The FFN and router weights depend on the group size only, so they are drawn once per group size
(their own seeded stream) and shared by the points of that size; the activations have their own
seeded stream per point.
"""
import functools

import numpy as np
import pytest
import torch

from oracle import wide_oracle as wo
from paper_2607_28418_b200 import synth
from tests.gpu_util import assert_all_rows_close, bits_to_host, ffn_ref_rows, to_dev

pytestmark = pytest.mark.gpu

GROUPS = (64, 128, 256)
FRACTIONS = (0.75, 0.5, 0.25)
# the clustered points alternate between the two prototype settings of the input recipe
PREFILL = [(G, p, r) for G in GROUPS for p in FRACTIONS for r in ("random", "clustered")]
DECODE = [(G, p, r) for G in GROUPS for p in FRACTIONS for r in ("random", "clustered_corr")]


@pytest.fixture(scope="module")
def ctx():
    from paper_2607_28418_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.status() == 0
    c.close()


@functools.lru_cache(maxsize=3)
def _weights(group: int):
    """Host and device copies of the 8B-shaped weights for one group size, kept for the points that share it."""
    cfg = synth.sweep_point(1, group, 0.5, "random")
    rng = np.random.default_rng(9000 + group)
    host = {
        "w_router": synth.make_weight(rng, cfg.n_groups, cfg.hidden, 1.0 / np.sqrt(cfg.hidden), "bf16"),
        "w_gate": synth.make_weight(rng, cfg.d_ff, cfg.hidden, 0.02, "bf16"),
        "w_up": synth.make_weight(rng, cfg.d_ff, cfg.hidden, 0.02, "bf16"),
        "w_down": synth.make_weight(rng, cfg.hidden, cfg.d_ff, 0.02, "bf16"),
    }
    return host, {k: to_dev(v, "bf16") for k, v in host.items()}


def _point(ctx, tokens, group, fraction, router):
    from paper_2607_28418_b200 import binding
    cfg = synth.sweep_point(tokens, group, fraction, router)
    host, dev = _weights(group)
    seed = 31 * tokens + group + int(100 * fraction) + len(router)
    x = synth.make_activations(np.random.default_rng(seed), tokens, cfg.hidden, "bf16", router)
    case = dict(host, x=x)
    xd = to_dev(x, "bf16")
    NG = cfg.n_groups
    bits, _ = binding.wide_route(ctx, xd, dev["w_router"], NG, cfg.k)
    mask = wo.mask_topk(wo.route_scores(x, host["w_router"]), cfg.k)
    assert (bits_to_host(bits) == wo.pack_mask_bits(mask)).all(), "mask bits differ"
    meta = None
    if tokens > 64:
        meta = binding.wide_reorder(ctx, bits, NG, 128)
        ref = wo.reorder(mask, 128)
        for name in ("perm", "counts", "tile_map", "offsets", "token_order", "token_rank"):
            assert (meta[name].cpu().numpy() == ref[name]).all(), name
        nw = int(meta["n_work"].item())
        assert nw == ref["n_work"] and (meta["work_list"].cpu().numpy()[:nw] == ref["work_list"]).all()
    y = binding.wide_ffn(ctx, xd, dev["w_gate"], dev["w_up"], dev["w_down"], group, bits, meta)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    assert_all_rows_close(y, ffn_ref_rows(case, mask, group), cfg.name)


@pytest.mark.parametrize("G,p,router", PREFILL)
def test_sweep_prefill_4096_tokens(ctx, G, p, router):
    _point(ctx, 4096, G, p, router)


@pytest.mark.parametrize("G,p,router", DECODE)
def test_sweep_decode_batch16(ctx, G, p, router):
    _point(ctx, 16, G, p, router)
