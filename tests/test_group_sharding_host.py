"""Host side of group sharding: the partition arithmetic, and -- on two gloo ranks -- that the parts
of Eq. 10's sum over groups, one group range per rank, all-reduce to the full result (CPU oracle on
both sides; no GPU)."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2607_28418_b200 import binding, synth  # noqa: E402


def test_group_ranges_tile_the_groups():
    for n_groups in (1, 7, 10, 86, 112, 224, 256):
        for world in (1, 2, 3, 4, 8):
            ranges = [binding.group_range(n_groups, world, r) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == n_groups
            for (a0, a1), (b0, b1) in zip(ranges, ranges[1:]):
                assert a1 == b0 and a0 <= a1
            sizes = [b - a for a, b in ranges]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)


def _rank(rank, world, port, out):
    import torch
    import torch.distributed as dist
    from oracle import wide_oracle as wo
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = synth.CONFIGS["tiny"]
    case = synth.make_ffn_case(cfg, 0, tokens=24)          # same seed on every rank: replicated inputs
    mask = wo.mask_topk(wo.route_scores(case["x"], case["w_router"]), cfg.k)   # routing is replicated
    g0, g1 = binding.group_range(cfg.n_groups, world, rank)
    c0, c1 = g0 * cfg.group, g1 * cfg.group
    part = wo.ffn(case["x"], case["w_gate"][c0:c1], case["w_up"][c0:c1], case["w_down"][:, c0:c1], mask[:, g0:g1], cfg.group)
    t = torch.from_numpy(part)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    full = wo.ffn(case["x"], case["w_gate"], case["w_up"], case["w_down"], mask, cfg.group)
    out.put((rank, float(np.abs(t.numpy() - full).max()), float(np.abs(full).max())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_all_reduce_their_group_ranges_to_the_full_result():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, 2, 29741, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=180) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, err, scale in got:
        assert err <= 1e-12 * scale
