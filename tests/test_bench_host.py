"""Host-side logic of bench.py (no GPU): work counts against closed forms and brute force, and the
multi-rank aggregation (replicas: max time over ranks, whole-job tokens/s) with two gloo ranks."""
import os
import subprocess
import sys
import textwrap

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2604_12452_b200 import inputs as I  # noqa: E402


def test_key_visits_matches_brute_force_and_the_quoted_counts():
    def brute(L, g, w):
        n = 0
        for t in range(1, L + 1):
            m_t = 0 if t < w + g else (t - w) // g
            n += m_t + (t - m_t * g)
        return n
    for L, g, w in [(1, 4, 0), (50, 64, 16), (300, 8, 64), (1000, 64, 128), (777, 16, 100)]:
        assert bench.key_visits(L, g, w) == brute(L, g, w)
    # counts quoted for the benchmark configurations (2176 flop per visit and head)
    assert abs(bench.key_visits(131072, 64, 4096) - 6.584e8) / 6.584e8 < 1e-3
    assert abs(bench.attention_flops(I.CONFIGS["mla_128k"]) - 183.4e12) / 183.4e12 < 1e-3
    assert abs(bench.attention_flops(I.CONFIGS["mla_32k"]) - 2.553e12) / 2.553e12 < 1e-3
    assert abs(bench.attention_flops(I.CONFIGS["gqa_64k"]) - 4.775e12) / 4.775e12 < 1e-3
    # window >= L is dense causal attention: L (L + 1) / 2 visits
    assert bench.key_visits(4096, 64, 4096) == 4096 * 4097 // 2


def test_condense_bytes_counts_every_stream_once():
    cfg = I.CONFIGS["mla_128k"]
    m, k = 1984, 4096
    expect = m * 64 * 1152 + 64 * 128 * 1152 + m * 1152 + 4 * m + 2 * k * 1152
    assert bench.condense_bytes(cfg) == expect


def test_two_gloo_ranks_report_the_slowest_time_and_the_whole_job_rate(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(textwrap.dedent(f"""
        import os, sys, json
        sys.path.insert(0, {ROOT!r})
        import torch, torch.distributed as dist
        import bench
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")      # rank 1 is slower
        value = bench.whole_job_value(131072, world, ms)
        if rank == 0:
            print(json.dumps(dict(ms=ms, value=value, world=world)))
        dist.destroy_process_group()
    """))
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["world"] == 2 and abs(line["ms"] - 15.0) < 1e-9
    assert abs(line["value"] - 2 * 131072 / 15e-3) < 1e-6


def test_gpus_flag_without_a_launcher_starts_one_rank_per_gpu():
    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "2"], port=29999)
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node=4" in cmd and "--nnodes=1" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1" and cmd[cmd.index("--master-port") + 1] == "29999"
    assert cmd[-5].endswith("bench.py") and cmd[-4:] == ["--gpus", "4", "--steps", "2"]
    # a free port is picked when none is given
    assert int(bench.launcher_command(2, [])[bench.launcher_command(2, []).index("--master-port") + 1]) > 0


def test_reference_arm_runs_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "mla_1k"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
