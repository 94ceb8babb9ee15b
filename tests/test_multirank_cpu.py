"""The N > 1 path of bench.py on CPU: two gloo ranks.

The method does not shard across GPUs (replicas only: every rank runs the same
independent batch, no data-path collective), so what N > 1 adds is the rank
plumbing: the timed region of the job is the slowest rank's (all-reduce MAX),
the reported value is the work of all ranks over that time, rank 0 alone
prints, and the reference arm does nothing on the other ranks.
"""
import io
import contextlib
import json
import os
import socket
import subprocess
import sys
import types

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 * (rank + 1)                     # rank 1 is the slow one
        total = bench.max_over_ranks(local_ms, world, "cpu")
        value = bench.whole_job_value(64, world, total)
        dist.barrier()
        # the reference arm: only rank 0 works and prints
        buf = io.StringIO()
        if rank != 0:
            with contextlib.redirect_stdout(buf):
                bench.run_reference(types.SimpleNamespace(config="tiny", steps=1, warmup=0), rank, world)
        with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
            json.dump(dict(total=total, value=value, ref_out=buf.getvalue()), f)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r in res:
        assert r["total"] == 20.0                         # max over ranks, the same on every rank
        assert abs(r["value"] - 2 * 64 / 0.020) < 1e-9    # units of all ranks / slowest time
    assert res[1]["ref_out"] == ""                        # rank 1 of the reference arm stays silent


def test_single_rank_needs_no_process_group():
    assert bench.max_over_ranks(7.5, 1, "cpu") == 7.5
    assert bench.whole_job_value(10, 1, 500.0) == 20.0


def test_reference_arm_line_on_the_tiny_config(capsys):
    """`--impl reference` prints one JSON line with the contract's keys (tiny config: seconds)."""
    bench.run_reference(types.SimpleNamespace(config="tiny", steps=1, warmup=0), 0, 1)
    line = json.loads(capsys.readouterr().out.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == bench.UNIT and line["higher_is_better"] is True
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"] > 0
    assert line["e2e"] == {"value": line["value"], "unit": bench.UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_gpus_flag_starts_the_ranks_itself():
    """`python bench.py --gpus 2` run as a plain process (no launcher, no WORLD_SIZE) must itself become two
    ranks.  `--plumbing-check` keeps the GPU work out: the ranks rendezvous over gloo on 127.0.0.1, take
    the slowest rank's time, and rank 0 alone prints the line, with n_gpus = 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, bench.__file__, "--gpus", "2", "--steps", "4", "--warmup", "3", "--plumbing-check"],
                         capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(l) for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                # rank 0 alone prints
    assert lines[0]["n_gpus"] == 2 and lines[0]["steps"] == 4
    assert abs(lines[0]["value"] - 2 * 4 / 0.020) < 1e-9  # work of both ranks over the slower rank's 20 ms


def test_gpus_flag_must_agree_with_the_launcher():
    env = dict(os.environ, WORLD_SIZE="1", RANK="0")
    res = subprocess.run([sys.executable, bench.__file__, "--gpus", "2", "--plumbing-check"], capture_output=True, text=True,
                         env=env, timeout=120)
    assert res.returncode == 2 and "disagrees" in res.stderr
