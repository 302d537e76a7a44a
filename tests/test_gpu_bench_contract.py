"""The benchmark's output contract, checked on a short run of the real thing (GPU)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_prints_one_json_line_with_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5", "--warmup", "3",
                          "--no-sweep", "--no-ablation", "--cpu-rows", "64", "--e2e-steps", "2"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    r = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e",
                "gpu_launches", "clocks", "per_kernel"):
        assert key in r, key
    assert r["n_gpus"] == 1 and r["steps"] == 5 and r["warmup"] == 3 and r["unit"] == "GB/s"
    assert r["higher_is_better"] is True and r["scaling"] == "weak" and r["vs_baseline"] is None
    assert r["dtype"] == "f32" and r["data"] == "synthetic" and "workload" in r["config"]
    assert r["gpu_launches"] == 6 * 5 + 3 * 2 * 4 and r["value"] > 1000.0  # + 2 end-to-end steps of 4 chunks
    rf = r["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and rf["peak"] > 0
    assert rf["frac"] == pytest.approx(rf["achieved"] / rf["peak"], rel=1e-3)
    assert rf["traffic"] is None or rf["traffic"] > 0
    cb = r["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] > 0 and cb["sample"]
    e = r["e2e"]
    assert e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and 0 < e["value"] < r["value"]
    assert set(r["per_kernel"]) == {"fused_add_rmsnorm", "silu_and_mul", "merge_attn_states_lse"}


def test_bench_started_plainly_with_two_ranks_spawns_them():
    """`python bench.py --gpus 2` without a launcher starts its own two ranks.  With one GPU in the
    machine the two ranks share it (gloo for the timing reduction; their kernels never wait on one
    another), which checks the multi-rank host path, not scaling."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--backend", "gloo",
                          "--steps", "3", "--warmup", "3", "--tokens", "512", "--e2e-steps", "1", "--no-clocks"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT, env=env)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["n_gpus"] == 2 and r["launcher"] == "self-spawned ranks" and r["scaling"] == "weak"
    assert "shape_sweep" not in r and "cpu_baseline" not in r   # rank-0-only extras are for the 1-GPU line
    assert r["value"] > 0 and r["config"]["tokens_per_gpu"] == 512
