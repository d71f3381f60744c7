"""Host-side logic of bench.py that needs no GPU: the max-over-ranks reduction of the replicas-only
multi-GPU mode (two gloo ranks on CPU), the whole-job value, the algorithmic-byte count and the
reference arm's rank handling."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_1712_01084_b200 import synth  # noqa: E402


def _rank_main(rank, world, port, q):
    import torch.distributed as dist
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow replica
    got = bench.max_over_ranks(ms, world, device="cpu")
    dist.barrier()
    q.put((rank, got))
    dist.destroy_process_group()


def test_max_over_ranks_two_gloo_ranks():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res == {0: 15.0, 1: 15.0}
    # two replicas, each one layer per 15 us step -> 7.5 us per layer for the job
    assert bench.job_value(15.0, 2) == 7.5 and bench.max_over_ranks(3.0, 1) == 3.0


def test_algorithmic_bytes_config5():
    wl = synth.config5(k=8, batch=1, scale=0.25)
    lay = wl.layers[0]
    n_tile_col = lay.Mb * 4                       # 2 tiles per block-row, padded to 4 entries
    got = bench.algorithmic_bytes(lay, 1, n_tile_col)
    want = lay.T * 64 * 64 * 2 + 4 * (n_tile_col + lay.Mb + 1) + lay.N * 2 + lay.M * 4 + 4 * (lay.N + lay.M)
    assert got == want


def test_tile_column_count_matches_the_packer():
    """bench.n_tile_col (per-block-row lists padded to 4 entries) is what the packer reports."""
    from paper_1712_01084_b200 import binding as pb
    wl = synth.config3(batch=1, scale=1 / 8)
    for lay in wl.layers:
        pk = pb.Packed(lay.M, lay.N, lay.B, lay.row_perm, lay.col_perm, lay.tile_list, lay.tile_values, lay.bias)
        assert bench.n_tile_col(lay) == pk.n_tile_col


def test_region_plan_covers_exactly_the_steps():
    for steps in (1, 20, 999, 1000, 1001, 2500, 20000):
        main, replays, rem = bench.region_plan(steps)
        assert main * replays + rem == steps and 0 < main <= bench.GRAPH_CALLS and 0 <= rem < main


def test_reference_arm_rank_handling():
    """Under a multi-rank launch only rank 0 runs the CPU oracle; the others exit 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--gpus", "2"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
