"""The multi-rank plumbing of bench.py on the CPU: two gloo ranks rendezvous, take the max of
their times, and only rank 0 reports.  (On GPUs the same code runs over NCCL, one rank per GPU,
each rank on its own column block: the update never mixes columns, so there is no collective on
the data path.)"""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, %(root)r)
import bench
rank, world, local_rank, dist = bench.dist_setup(2)
assert world == 2 and dist is not None and rank == int(os.environ["RANK"])
ms = 10.0 + 5.0 * rank            # rank 1 is the slow one
dist.barrier()
slowest = bench.max_over_ranks(ms, dist, "cpu")
units = 1000
value = world * units / (slowest * 1e-3)
if rank == 0:
    print(json.dumps({"slowest_ms": slowest, "value": value, "world": world}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, extra_env):
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="", **extra_env)
        procs.append(subprocess.Popen([sys.executable] + code_or_args, env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True, cwd=ROOT))
    outs = [p.communicate(timeout=240) for p in procs]
    for p, (out, err) in zip(procs, outs):
        assert p.returncode == 0, err[-2000:]
    return [o for o, _ in outs]


def test_two_gloo_ranks_report_the_slowest_time_once():
    outs = _spawn(["-c", WORKER % {"root": ROOT}], {})
    assert outs[1].strip() == ""                      # only rank 0 prints
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["world"] == 2 and line["slowest_ms"] == 15.0
    assert abs(line["value"] - 2 * 1000 / 15e-3) < 1e-6


def test_reference_arm_runs_on_rank_zero_only():
    outs = _spawn([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2", "--warmup", "1",
                   "--workload", "step_small"], {"OMP_NUM_THREADS": "2"})
    assert outs[1].strip() == ""
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0
