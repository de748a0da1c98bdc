"""The multi-rank plumbing of bench.py on CPU (gloo, world size 2): replicas only, so all
there is to check is the max-over-ranks timing, the whole-job aggregate and that the
reference arm prints on rank 0 alone."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch.distributed as dist
import bench
dist.init_process_group("gloo", init_method="tcp://127.0.0.1:%%s" %% os.environ["PORT"],
                        rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank = dist.get_rank()
mine = 1.0 + 2.0 * rank                      # rank 0: 1 s, rank 1: 3 s
slowest = bench.max_over_ranks(mine, dist, "cpu")
dist.barrier()
print("RESULT %%d %%.3f %%.3f" %% (rank, slowest, bench.whole_job_value(10.0, 6, dist.get_world_size(), slowest)))
dist.destroy_process_group()
""" % ROOT


def _free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks():
    port = str(_free_port())
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", PORT=port)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    for rank, (out, _) in enumerate(outs):
        line = [l for l in out.splitlines() if l.startswith("RESULT")][0].split()
        assert int(line[1]) == rank
        assert float(line[2]) == 3.0                     # both ranks see the slowest rank's time
        assert float(line[3]) == 2 * 10.0 * 6 / 3.0      # two replicas' units over that time


def test_single_process_helpers_need_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(0.25, None, "cpu") == 0.25
    assert bench.whole_job_value(4.0, 5, 1, 2.0) == 10.0


def test_reference_arm_prints_on_rank_zero_only():
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--steps", "2", "--warmup", "1"]
    env1 = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    r1 = subprocess.run(cmd, env=env1, capture_output=True, text=True, timeout=600)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    env0 = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="2")
    r0 = subprocess.run(cmd, env=env0, capture_output=True, text=True, timeout=600)
    assert r0.returncode == 0, r0.stderr[-2000:]
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["unit"] == "GB/s" and line["higher_is_better"] is True
    sys.path.insert(0, ROOT)
    import bench
    # both arms name the workload with the same string (the driver compares them)
    assert line["config"]["workload"] == bench.workload_name(bench.w.CONFIGS[bench.HEADLINE])
    assert line["metric"] == bench.METRIC


def test_gpus_n_without_a_launcher_environment_starts_the_ranks_itself():
    sys.path.insert(0, ROOT)
    import bench
    cmd = bench.rank_command(2, ["--gpus", "2", "--steps", "3"])
    assert cmd[1:3] == ["-m", "torch.distributed.run"] and "--nproc-per-node" in cmd
    assert cmd[cmd.index("--nproc-per-node") + 1] == "2" and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[-4:] == ["--gpus", "2", "--steps", "3"] and cmd[-5].endswith("bench.py")
    # end to end on CPU through the reference arm: two ranks are started, rank 0 alone prints
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE")}
    run = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=900)
    assert run.returncode == 0, run.stderr[-2000:]
    lines = [l for l in run.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2


def test_loop_count_and_spread():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.loop_count(0.25e-3) == 200            # blocks of 0.25 ms: 200 of them make 50 ms
    assert bench.loops_per_block(20) == 10 and bench.loops_per_block(1000) == 1 and bench.loops_per_block(7) == 29
    assert bench.loop_count(1.0) == bench.MIN_LOOPS      # long loops: the minimum number of repeats
    assert bench.loop_count(1e-9) == bench.MAX_LOOPS
    s = bench.spread([2e-4, 1e-4, 4e-4], 10)
    assert s["us_per_step_median"] == pytest.approx(20.0) and s["us_per_step_min"] == pytest.approx(10.0)
    assert s["us_per_step_max"] == pytest.approx(40.0) and s["loops"] == 3
    assert bench.workload_name(bench.w.CONFIGS[1]).startswith("cfg2_gemv b,m,k,n=[1, 1, 2048, 16384]")
