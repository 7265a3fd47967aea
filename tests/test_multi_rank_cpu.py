"""The N > 1 path of bench.py on CPU (gloo, world size 2): replicas only, so what has to hold is
that ranks draw different inputs, that every rank reports the slowest rank's time, that the
aggregate counts all ranks' tokens, and that the reference arm works on rank 0 alone."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2604_22808_b200 import configs as C  # noqa: E402
from paper_2604_22808_b200 import inputs as I  # noqa: E402


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = bench.replica_config(C.TINY, rank)
    x = I.qkv_head(cfg, 0, 0, 0)
    ms_local = 1.0 + rank                                   # rank 1 is the slow one
    ms = bench.reduce_max(ms_local, world, "cpu")
    dist.barrier()
    out.put((rank, float(x.reshape(-1)[0]), ms, bench.aggregate_tokens_per_s(C.TINY, world, ms)))
    dist.destroy_process_group()


def test_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29533, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (r0, x0, ms0, v0), (r1, x1, ms1, v1) = res
    assert x0 != x1                                         # each rank its own replica
    assert ms0 == ms1 == 2.0                                # slowest rank's time everywhere
    assert v0 == v1 == 2 * C.TINY.batch * C.TINY.N / 2e-3   # all ranks' tokens over that time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_fp32",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_fp32",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0
    import json
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0


def test_forced_allocation_option():
    """`--alloc L,M,H`: heads [0,L) low, the next M mid, the rest high, repeated per sample."""
    cfg = C.G128K                                   # batch 2, 24 heads
    masks = bench.forced_allocation(cfg, "12,8,4")
    assert len(masks) == cfg.batch * cfg.heads
    assert masks[:24] == [1] * 12 + [2] * 8 + [4] * 4 and masks[24:] == masks[:24]
    assert bench.forced_allocation(cfg, "") is None
    for bad in ("12,8", "12,8,5", "-1,13,12"):
        try:
            bench.forced_allocation(cfg, bad)
        except SystemExit:
            continue
        raise AssertionError(f"--alloc {bad} was accepted")


def test_layer_work_counts_follow_the_cost_formulas():
    """bench.py's interaction counts (its useful-FLOP figure) equal the oracle's counters."""
    from oracle import freqformer_oracle as O
    for cfg in (C.TINY, C.G64K, C.R1M, C.PAPER_REF_64K):
        sizes = [len(x) for x in O.band_members(cfg.grid, cfg.low_cut, cfg.mid_cut)]
        n_bar = -(-sizes[0] // cfg.r)
        expect = (n_bar * n_bar, O.mid_interactions(sizes[1], cfg.b, cfg.s), O.high_interactions(sizes[2], cfg.R))
        assert bench.interactions(cfg) == expect, (cfg.name, bench.interactions(cfg), expect)
        alloc = [1, 2, 4, 7][: cfg.heads] * cfg.batch
        work = bench.layer_work(cfg, alloc)
        per_mask = {1: expect[0], 2: expect[1], 4: expect[2], 7: sum(expect)}
        assert work["attn_flops"] == 4 * cfg.head_dim * sum(per_mask[m] for m in alloc)
