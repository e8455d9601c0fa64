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


SHARD_WORKER = r"""
import os, sys, json
sys.path.insert(0, %(root)r)
import numpy as np, torch, torch.distributed as dist
import bench, oracle, synthetic_inputs as synth
from paper_2306_00256_b200 import shard_columns
rank, world, local_rank, d_ = bench.dist_setup(2)
n, m, d, k = 6, 40, 1030, 1
a, lab, _ = synth.logreg_problem(n, m, d, seed=11, flip=0.1, hetero_std=0.5)      # every rank draws the same problem
gen = torch.Generator().manual_seed(12)
x, y = 0.1 * torch.randn(n, d, generator=gen), 0.1 * torch.randn(n, d, generator=gen)
z = y if oracle.round_info(n, k).payload else x
lo, hi = shard_columns(d, world, rank)
# (i) partial dot products of this rank's column block, (ii) their sum over the ranks
dots = torch.einsum("nmc,nc->nm", a[:, :, lo:hi].double(), z[:, lo:hi].double())
dist.all_reduce(dots, op=dist.ReduceOp.SUM)
# (iii) coefficient per sample, then this block's columns of the gradient
coef = -(lab.double() / m) / (1.0 + torch.exp(lab.double() * dots))
g_block = torch.einsum("nm,nmc->nc", coef, a[:, :, lo:hi].double())
want = oracle.logreg_grad(a.numpy(), lab.numpy(), x.numpy(), y.numpy(), k)[:, lo:hi]
err = float(np.abs(g_block.numpy() - want).max())
widths = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
dist.all_gather(widths, torch.tensor([hi - lo]))
if rank == 0:
    print(json.dumps({"err": err, "widths": [int(w) for w in widths], "d": d}))
assert err < 1e-12
dist.destroy_process_group()
"""


def test_column_sharded_gradient_over_two_gloo_ranks():
    """The rank plumbing of the column-sharded gradient on the CPU: each rank holds a column block, the
    n x m partial dot products are summed with one all-reduce, and each rank's gradient block equals the
    oracle's columns.  (On GPUs the three steps are dsgd_grad_shard_dots, an NCCL all-reduce and
    dsgd_grad_shard_apply; the arithmetic here is plain torch on the CPU, standing in for the kernels.)"""
    outs = _spawn(["-c", SHARD_WORKER % {"root": ROOT}], {"OMP_NUM_THREADS": "2"})
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert sum(line["widths"]) == line["d"] and all(w % 4 == 0 for w in line["widths"][:-1])
    assert line["err"] < 1e-12
