"""Host-side logic of bench.py (no GPU): the byte model, the replica seeding, the max-over-ranks reduction on two
gloo ranks, and the CPU-oracle arm (--impl reference) including its behaviour under a two-rank launch."""
import json
import os
import subprocess
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2201_12667_b200 import workloads  # noqa: E402


def test_byte_model_counts_each_distinct_row_once_per_use():
    c = workloads.config("670k")
    per = dict(nnz=19500.0, sum_active=35500.0, touched_w1=7200.0, touched_w2=32000.0, fetched=34300.0)
    m = bench.byte_model(c, 256, per, 1280.0, 50)
    H, N, L = c["H"], c["N"], c["L"]
    w1 = 6 * 4 * H * 7200
    w2 = 6 * 4 * (H + 1) * 32000
    assert m["adam"] == pytest.approx(w1 + w2 + 24 * H + 8 * 35500 + 4 * 256 * H)
    rebuild = (4 * H * N + 4 * N * L + 4 * L * (2 ** 18 + 1)) / 50
    assert m["rebuild"] == pytest.approx(rebuild)
    # the forward kernel's own figure adds the rows it gathers; the step total counts every distinct row once
    gathered = 4 * H * 19500 + 4 * (H + 1) * 35500
    assert m["total"] == pytest.approx(m["adam"] + m["forward"] - gathered + rebuild)
    # no rebuild scheduled -> no rebuild bytes
    assert bench.byte_model(c, 256, per, 1280.0, 0)["rebuild"] == 0.0
    assert bench.code_bits(workloads.config("325k")) == 9 and bench.code_bits(c) == 18


def test_replicas_draw_different_batches():
    c = workloads.config("mid")
    a = workloads.Workload(c, seed=bench.shard_seed(0)).batch(0)
    b = workloads.Workload(c, seed=bench.shard_seed(1)).batch(0)
    assert not np.array_equal(a[1][:20], b[1][:20])


_RANK_SCRIPT = """
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
world, rank, local = bench.dist_setup(2)
dist.init_process_group("gloo", rank=rank, world_size=world)
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")
dist.barrier()
dist.destroy_process_group()
print("RESULT", rank, world, ms)
"""


def test_max_over_ranks_on_two_gloo_ranks(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT % ROOT)
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT="29671")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    for r, (out, err) in enumerate(outs):
        assert procs[r].returncode == 0, err[-2000:]
        line = [x for x in out.splitlines() if x.startswith("RESULT")][0].split()
        assert int(line[1]) == r and int(line[2]) == 2 and float(line[3]) == 15.0     # the slower rank's time on both


def test_reference_arm_prints_one_json_line_and_only_on_rank_zero():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "tiny", "--steps", "3",
           "--warmup", "1", "--gpus", "2"]
    env0 = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    out = subprocess.run(cmd, env=env0, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [x for x in out.stdout.splitlines() if x.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["unit"] == "samples/s" and d["value"] > 0 and d["steps"] == 3
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "samples/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["vs_baseline"] is None and d["higher_is_better"] is True and d["dtype"] == "f32"
    env1 = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out1 = subprocess.run(cmd, env=env1, capture_output=True, text=True, timeout=600)
    assert out1.returncode == 0 and out1.stdout.strip() == ""


def test_full_step_accounting_never_drops_or_doubles_the_rebuild():
    # 500 steps at period 50 with the 10 scheduled rebuilds inside: as measured
    ms, how = bench.full_step_ms(40.0, 500, 10, 0.9, 50)
    assert ms == pytest.approx(0.08) and how.startswith("as measured")
    # 20 steps without any rebuild inside: one rebuild per 50 steps is added
    ms, how = bench.full_step_ms(1.2, 20, 0, 0.9, 50)
    assert ms == pytest.approx(1.2 / 20 + 0.9 / 50) and "added per 50 steps" in how
    # 30 steps that happen to hold one rebuild (1 per 30 > 1 per 50): taken out, then charged at 1 per 50
    ms, _ = bench.full_step_ms(30 * 0.06 + 0.9, 30, 1, 0.9, 50)
    assert ms == pytest.approx(0.06 + 0.9 / 50)
    # no schedule
    assert bench.full_step_ms(2.0, 20, 0, 0.0, 0)[0] == pytest.approx(0.1)


def test_sweep_grid_covers_the_batch_and_fraction_axes():
    assert bench.SWEEP_BATCHES == (64, 128, 256, 512, 1024, 2048)
    fr = [f for f, _ in bench.SWEEP_FRACTIONS]
    assert fr[0] == 0.0005 and fr[-1] == 1.0 and bench.SWEEP_FRACTIONS[-1][1] == dict(force_dense=1)
    N = workloads.config("670k")["N"]
    for f, over in bench.SWEEP_FRACTIONS[:-1]:
        per_bucket = min(over["bucket_cap"], N / 8 ** over["K"])
        assert 0.6 * f * N <= over["L"] * per_bucket <= 1.7 * f * N      # duplicates shrink the union of large buckets
