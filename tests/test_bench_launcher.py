"""`bench.py --gpus N` as N ranks: the launcher, rank discovery, distinct per-rank stream scripts over one shared
corpus, the reduction and the single JSON line - on two gloo ranks with the step stubbed out - and the reference
arm over the same rank shares.  CPU only."""
from __future__ import annotations

import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
import workload as W  # noqa: E402
from harness.launcher import launch_command, spawn_ranks  # noqa: E402

STUB = os.path.join(ROOT, "tests", "launcher_stub_rank.py")
ARGS = ["--config", "0", "--steps", "3", "--warmup", "3", "--split-steps", "0", "--e2e-steps", "0", "--cpu-steps", "4"]


def _json_lines(text):
    return [json.loads(ln) for ln in text.splitlines() if ln.startswith("{")]


def test_two_ranks_one_line():
    rc, out, err = spawn_ranks(2, STUB, ["--gpus", "2", *ARGS], capture=True, timeout=300)
    assert rc == 0, err[-2000:]
    lines = _json_lines(out)
    assert len(lines) == 1, out
    d = lines[0]
    cfg = W.CONFIGS[0]
    assert d["n_gpus"] == 2 and d["scaling"] == "weak" and d["steps"] == 3 and d["warmup"] == 3
    assert d["local_ranks"] == [0, 1]
    # tokens are summed over ranks, time is the slowest rank's
    assert abs(d["value"] - (cfg.B * 3 * (1 + 2)) / 0.020) < 1e-6
    assert abs(d["ms_per_step"] - 20.0 / 3) < 1e-9
    # every rank owns streams of its own over the one replicated corpus
    assert d["rank_seeds"] == [cfg.seed, cfg.seed + bench.RANK_SEED_STRIDE]
    assert len(set(d["script_digests"])) == 2 and len(set(d["corpus_digests"])) == 1
    assert d["config"]["workload"] == cfg.name and d["config"]["B_per_gpu"] == cfg.B


def test_world_size_must_match_gpus():
    rc, out, err = spawn_ranks(2, STUB, ["--gpus", "3", *ARGS], capture=True, timeout=300)
    assert rc != 0
    assert "launcher started 2 rank" in err
    assert _json_lines(out) == []


def test_launch_command_is_the_documented_one():
    cmd = launch_command(4, "bench.py", ["--gpus", "4"], port=29511)
    assert cmd[1:] == ["-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=4", "--master-addr", "127.0.0.1",
                       "--master-port", "29511", "bench.py", "--gpus", "4"]


def test_reference_arm_covers_every_rank_share():
    """--impl reference --gpus 2 in one process: the oracle over both rank shares, same config block and the same
    per-rank seeds as the GPU arm would use."""
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", *ARGS],
                       capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert p.returncode == 0, p.stderr[-2000:]
    (d,) = _json_lines(p.stdout)
    one = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "1", *ARGS],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    (d1,) = _json_lines(one.stdout)
    cfg = W.CONFIGS[0]
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d1["n_gpus"] == 1
    assert d["steps"] == 3 and d["warmup"] == 3
    assert d["rank_seeds"] == [cfg.seed, cfg.seed + bench.RANK_SEED_STRIDE] and d1["rank_seeds"] == [cfg.seed]
    args = bench.parse_args(["--gpus", "2", *ARGS])
    assert d["config"] == bench.workload_block(bench.plan_rank(args, 0)[0]) == d1["config"]
    assert d["e2e"]["value"] == d["value"] and d["cpu_baseline"]["kind"] == "oracle"
    assert d["gpu_launches"] == 0
