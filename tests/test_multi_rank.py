"""world_size-2 checks of the multi-process host logic on CPU (gloo): row sharding, the
max-over-ranks timing reduction, and the benchmark's reference arm under torchrun."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_07506_b200 import multi

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_rows_partition():
    for total in (0, 1, 2, 7, 8, 8192, 8193, 16383):
        for world in (1, 2, 3, 4, 8):
            seen = []
            for rank in range(world):
                first, count = multi.shard_rows(total, world, rank)
                seen.extend(range(first, first + count))
                assert count in (total // world, total // world + 1)
            assert seen == list(range(total))
    with pytest.raises(ValueError):
        multi.shard_rows(8, 2, 2)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    multi.init_process_group("gloo")
    try:
        assert multi.env_rank_world() == (rank, world, rank)
        # every rank reports its own times; all must end up with the elementwise maximum
        mine = [10.0 + rank, 5.0 - rank, 1.0]
        got = multi.max_over_ranks(mine)
        assert got == [10.0 + world - 1, 5.0, 1.0]
        # shards of one batch: gather the row indices every rank owns and check the cover on rank 0
        first, count = multi.shard_rows(1001, world, rank)
        owned = torch.zeros(1001, dtype=torch.int32)
        owned[first:first + count] = 1
        dist.all_reduce(owned)
        assert bool((owned == 1).all())
        rate = multi.aggregate_rate(100.0, world, steps=4, elapsed_ms=got[0])
        assert rate == pytest.approx(world * 100.0 * 4 / (got[0] * 1e-3))
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as fh:
            fh.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    port = 29600 + os.getpid() % 300
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "ok0").exists() and (tmp_path / "ok1").exists()


def test_reference_arm_under_torchrun_prints_one_line():
    port = 29900 + os.getpid() % 90
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2",
           "--warmup", "3", "--cpu-rows", "32"]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["gpu_launches"] == 0
    assert rec["cpu_baseline"]["kind"] == "oracle" and rec["cpu_baseline"]["value"] == rec["value"]
    assert rec["e2e"]["h2d_bytes_per_step"] == 0 and rec["e2e"]["d2h_bytes_per_step"] == 0
