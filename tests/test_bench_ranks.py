"""The benchmark's N > 1 logic on CPU: two gloo ranks, no GPU.

The path does not shard ("replicas only"), so what the ranks share is small: disjoint episode numbers, the
max-over-ranks of the device times, the whole-job metric, and the rule that the reference arm runs on rank 0 alone.
"""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
import bench
world, rank, local = bench.rank_env()
dist.init_process_group("gloo", rank=rank, world_size=world)
B = 3
mine = bench.episodes_of_rank(rank, B)
# every rank reports its own (fake) device times; the job's time is the slowest rank's
times = [10.0 + 5.0 * rank, 40.0 - 7.0 * rank]
agg = bench.max_over_ranks(times, world)
gathered = [None] * world
dist.all_gather_object(gathered, mine)
dist.barrier()
print(json.dumps({"rank": rank, "world": world, "episodes": mine, "all": gathered, "agg": agg,
                  "metric": bench.job_us_per_step(agg[0], steps=4, world=world, B=B)}))
dist.destroy_process_group()
"""


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch(world, argv, extra_env=None):
    port = free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        env.update(extra_env or {})
        procs.append(subprocess.Popen([sys.executable] + argv, env=env, cwd=ROOT, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=280)
        outs.append((p.returncode, out, err))
    return outs


@pytest.mark.timeout(300)
def test_two_gloo_ranks_shard_episodes_and_take_the_slowest_time():
    outs = launch(2, ["-c", WORKER, ROOT])
    recs = []
    for rc, out, err in outs:
        assert rc == 0, err[-2000:]
        recs.append(json.loads(out.strip().splitlines()[-1]))
    recs.sort(key=lambda r: r["rank"])
    assert [r["world"] for r in recs] == [2, 2]
    assert recs[0]["episodes"] == [0, 1, 2] and recs[1]["episodes"] == [3, 4, 5]
    assert recs[0]["all"] == recs[1]["all"] == [[0, 1, 2], [3, 4, 5]]          # disjoint, and together 0..5
    for r in recs:
        assert r["agg"] == [15.0, 40.0]                                          # max over ranks, element-wise
        # 4 steps x 2 ranks x 3 episodes in 15 ms -> 625 us per episode-step, whole job
        assert abs(r["metric"] - 15.0e3 / (4 * 2 * 3)) < 1e-9


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.0, 1.0], world=1) == [3.0, 1.0]
    assert bench.episodes_of_rank(0, 1) == [0]
    assert bench.job_us_per_step(2.0, steps=4, world=1, B=1) == 500.0


@pytest.mark.timeout(300)
def test_reference_arm_runs_on_rank_zero_alone():
    """Launched as two ranks, rank 0 times the oracle and prints the line, rank 1 exits 0 without output."""
    outs = launch(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                      "--workload", "config1"])
    (rc0, out0, err0), (rc1, out1, err1) = outs
    assert rc0 == 0, err0[-2000:]
    assert rc1 == 0 and out1.strip() == ""
    line = json.loads(out0.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
