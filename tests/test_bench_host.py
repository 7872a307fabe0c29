"""Host-side logic of bench.py: workload selection, throughput aggregation, the max-over-ranks
reduction (two gloo ranks on CPU), and the shape of the reference arm's JSON line."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402


class _Args:
    workload = "llama7b_prefill"
    batch = 0
    router = ""
    k = None
    group = 0


def test_default_workload_is_the_7b_prefill_config():
    cfg = bench.make_config(_Args())
    assert (cfg.tokens, cfg.hidden, cfg.d_ff, cfg.group, cfg.n_groups, cfg.k) == (2048, 4096, 11008, 128, 86, 43)


def test_overrides_keep_the_active_fraction():
    a = _Args()
    a.workload, a.group, a.batch, a.router = "llama8b_prefill", 64, 16, "clustered"
    cfg = bench.make_config(a)
    assert cfg.n_groups == 224 and cfg.k == 112 and cfg.tokens == 16 and cfg.router == "clustered"


def test_aggregate_counts_all_ranks():
    # 4 ranks x 2048 tokens x 10 steps in 5 ms (max over ranks)
    assert bench.aggregate(2048, 10, 5.0, 4) == 4 * 2048 * 10 / 5e-3
    assert bench.flops_ffn_active(bench.make_config(_Args())) == 6.0 * 2048 * 43 * 128 * 4096


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.reduce_max_ms(10.0 + 5.0 * rank, world)      # rank 1 is slower
    value = bench.aggregate(2048, 4, ms, world)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, ms, value))


def test_max_over_ranks_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29731, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, ms, value in got:
        assert ms == 15.0                                    # both ranks see the slower rank's time
        assert value == 2 * 2048 * 4 / 15e-3


def test_reference_arm_prints_one_json_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--workload", "tiny"], capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    # under torchrun every rank but 0 exits without work
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny"],
                       capture_output=True, text=True, timeout=120, env=env)
    assert r.returncode == 0 and r.stdout.strip() == ""
