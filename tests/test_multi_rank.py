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


def _tp_worker(rank, world, port, out_dir):
    """The pointer-exchange logic of the fused all-reduce, with CPU tensors standing in for device
    buffers: handles are (owner, file) pairs, 'opening' one reads the owner's file."""
    import numpy as np
    import oracle
    from paper_2509_07506_b200 import workloads as wl
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    multi.init_process_group("gloo")
    try:
        T, H = 10, 48
        inp = wl.allreduce_rmsnorm_inputs(T, H, world, wl.BF16, seed=5)   # same seed: every rank knows all partials
        mine = inp.parts[rank]
        opened = []

        def export(t):
            path = os.path.join(out_dir, f"partial{rank}.pt")
            torch.save(t, path)
            return (rank, path)

        def open_remote(handle, owner):
            assert handle[0] == owner and owner != rank      # own slot must not be re-opened
            opened.append(owner)
            return torch.load(handle[1])

        parts = multi.exchange_partials(mine, export, open_remote)
        assert len(parts) == world and parts[rank] is mine and sorted(opened) == [r for r in range(world) if r != rank]
        for owner in range(world):
            assert torch.equal(parts[owner], inp.parts[owner]), "partials are not in rank order"
        # every rank normalises its own row block from all partials; together they cover the batch,
        # and each block equals the corresponding rows of the whole-batch result (rows are independent)
        first, count = multi.row_block_of_rank(T)
        sl = slice(first, first + count)
        y, r = oracle.fused_allreduce_add_rmsnorm([wl.bits(p[sl]) for p in parts], wl.bits(inp.residual[sl]),
                                                  wl.bits(inp.weight), inp.eps, wl.BF16)
        yw, rw = oracle.fused_allreduce_add_rmsnorm([wl.bits(p) for p in inp.parts], wl.bits(inp.residual),
                                                    wl.bits(inp.weight), inp.eps, wl.BF16)
        assert np.array_equal(y, yw[sl]) and np.array_equal(r, rw[sl])
        owned = torch.zeros(T, dtype=torch.int32)
        owned[sl] = 1
        dist.all_reduce(owned)
        assert bool((owned == 1).all())
        # Two-shot form, host side: every rank's output buffer is exchanged the same way (here a file
        # mapped by both processes stands for peer-mapped device memory), every rank stores its block
        # into all of them, and after a barrier each rank holds the whole-batch result.
        def export_map(arr):
            return (rank, arr.filename)

        def open_map(handle, owner):
            assert handle[0] == owner and owner != rank
            return np.memmap(handle[1], dtype=np.float64, mode="r+", shape=(T, H))

        y_mine = np.memmap(os.path.join(out_dir, f"y{rank}.bin"), dtype=np.float64, mode="w+", shape=(T, H))
        y_mine[:] = -1.0
        y_mine.flush()
        ys = multi.exchange_buffers(y_mine, export_map, open_map)
        assert len(ys) == world and ys[rank] is y_mine
        dist.barrier()
        for dest in ys:
            dest[sl] = y
            dest.flush()
        dist.barrier()
        assert np.array_equal(np.asarray(y_mine), yw), "two-shot: the assembled rows differ from the whole-batch result"
        with open(os.path.join(out_dir, f"tp_ok{rank}"), "w") as fh:
            fh.write("ok")
    finally:
        dist.destroy_process_group()


def test_partial_exchange_two_ranks_gloo(tmp_path):
    mp.spawn(_tp_worker, args=(2, multi.free_port(), str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "tp_ok0").exists() and (tmp_path / "tp_ok1").exists()


def test_exchange_partials_without_a_process_group_is_the_local_buffer():
    t = torch.zeros(3)
    assert multi.exchange_partials(t, None, None) == [t] and multi.row_block_of_rank(7) == (0, 7)


def test_spawn_ranks_gives_each_rank_its_environment(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(
        "import os, sys\n"
        "r, w = os.environ['RANK'], os.environ['WORLD_SIZE']\n"
        "assert os.environ['LOCAL_RANK'] == r and os.environ['MASTER_ADDR'] == '127.0.0.1'\n"
        "open(os.path.join(sys.argv[1], 'seen' + r), 'w').write(w + ' ' + os.environ['MASTER_PORT'])\n"
        "sys.exit(3 if (len(sys.argv) > 2 and r == '1') else 0)\n")
    assert multi.spawn_ranks([sys.executable, str(script), str(tmp_path)], 3) == 0
    seen = [(tmp_path / f"seen{r}").read_text().split() for r in range(3)]
    assert all(s[0] == "3" for s in seen) and len({s[1] for s in seen}) == 1
    assert multi.spawn_ranks([sys.executable, str(script), str(tmp_path), "fail"], 2) == 3


def test_reference_arm_started_without_a_launcher_reports_all_gpus():
    """`python bench.py --gpus 2` (no torchrun): the benchmark starts its own ranks; one JSON line."""
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2",
           "--warmup", "3", "--cpu-rows", "32"]
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["impl"] == "reference" and rec["n_gpus"] == 2 and rec["launcher"] == "self-spawned ranks"


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
