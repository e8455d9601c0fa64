#!/usr/bin/env python
"""Benchmark of the DSGD-CECA hot path: fused SGD step + one CECA gossip round per iteration.

Default workload ("resnet50_step"): n = 100 agents, d = 25,557,032 parameters per agent (a
ResNet-50-sized flat vector), fp32, CECA-2P, X0 = Y0 ~ N(0, 0.01^2), G ~ N(0, 0.01^2), gamma = 0.1,
updated in place.  A step is one call of ceca_gossip_sgd_step for iteration k (k keeps counting,
so the steps cycle through all tau = 7 rounds of the CECA sequence).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line (rank 0).  `value` is agent-parameter updates per second summed over all
ranks, inputs resident in HBM; `e2e` is the same metric through ceca_gossip_sgd_step_host with
pinned HOST buffers (copies inside the timed region); `roofline` is the dominant kernel's
algorithmic bytes over its CUDA-event time against the measured copy bandwidth;
`cpu_baseline` is the fp64 oracle timed on the host cores on a column slice.

With N > 1 (torchrun) every rank runs the same workload on its own GPU: the update never mixes
columns, so ranks are independent column blocks and there is no collective on the data path.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "agent-param updates/s (n*d per gossip+SGD step)"
UNIT = "agent-param updates/s"

# name -> (kind, n, d, variant, extra)
WORKLOADS = {
    # the configuration the headline metric is quoted on
    "resnet50_step": dict(kind="step", n=100, d=25_557_032, variant=2, gamma=0.1),
    # the same, but the caller declines the dead y+ of the last round of each cycle (one write less in 1 of 7 steps)
    "resnet50_step_dead_y": dict(kind="step", n=100, d=25_557_032, variant=2, gamma=0.1, drop_dead_y=True),
    # narrower storage, fp32 arithmetic (not in the paper): G as bf16 (18 B per agent-parameter), or X, Y, G as bf16 (10 B)
    "resnet50_step_g_bf16": dict(kind="step", n=100, d=25_557_032, variant=2, gamma=0.1, storage="g_bf16"),
    "resnet50_step_bf16": dict(kind="step", n=100, d=25_557_032, variant=2, gamma=0.1, storage="bf16"),
    # smaller cases of the same kernels, for profiler captures and quick looks
    "resnet18_step": dict(kind="step", n=24, d=11_689_512, variant=1, gamma=0.1),
    "step_small": dict(kind="step", n=100, d=2_097_152, variant=2, gamma=0.1),
    # rows a multiple of 4 floats apart, but X, Y and G all start one float past a 16-byte boundary (views that
    # skip the first element of their buffers): a scalar head of 3 columns, then the 128-bit body
    "step_offset_base": dict(kind="step", n=100, d=4_194_300, variant=2, gamma=0.1, base_offset=1),
    # nothing to align: ld = d = 4,194,303, every column runs the scalar form
    "step_odd_ld": dict(kind="step", n=100, d=4_194_303, variant=2, gamma=0.1, ld=4_194_303),
    # n a power of two: the X-only update (12 B per agent-parameter; CECA-2P = one-peer exponential graph)
    "pow2_xonly_step": dict(kind="step", n=128, d=8_388_608, variant=2, gamma=0.1, x_only=True),
    # fused = 1 picks the kernel by n and variant (register blocks for CECA-2P up to n = 1152 and CECA-1P up to n = 416)
    "consensus_fused": dict(kind="consensus", n=97, d=1 << 20, variant=2, fused=1),
    "consensus_fused_smem": dict(kind="consensus", n=97, d=1 << 20, variant=2, fused=2),
    "consensus_fused_tmem": dict(kind="consensus", n=97, d=1 << 20, variant=2, fused=3),
    "consensus_rounds": dict(kind="consensus", n=97, d=1 << 20, variant=2, fused=0),
    # the 1-port sequence (pairwise exchange, even n): fused and per round
    "consensus_fused_1p": dict(kind="consensus", n=100, d=1 << 20, variant=1, fused=1),
    "consensus_rounds_1p": dict(kind="consensus", n=100, d=1 << 20, variant=1, fused=0),
    "consensus_fused_1p_258": dict(kind="consensus", n=258, d=1 << 19, variant=1, fused=1),
    "consensus_fused_1p_258_smem": dict(kind="consensus", n=258, d=1 << 19, variant=1, fused=2),
    # half the columns: the case the profiler captures are taken on (0.2 GB in, 0.4 GB out)
    "consensus_fused_small": dict(kind="consensus", n=97, d=1 << 19, variant=2, fused=1),
    # the paper's network sizes (Sec. 5): n = 130, n = 258 (32-column tiles) and n = 1026 (16-column tiles, eleven rounds)
    "consensus_fused_130": dict(kind="consensus", n=130, d=1 << 20, variant=2, fused=1),
    "consensus_fused_258": dict(kind="consensus", n=258, d=1 << 19, variant=2, fused=1),
    "consensus_fused_1026": dict(kind="consensus", n=1026, d=1 << 18, variant=2, fused=1),
    "consensus_fused_1026_smem": dict(kind="consensus", n=1026, d=1 << 18, variant=2, fused=2),
    "consensus_rounds_1026": dict(kind="consensus", n=1026, d=1 << 18, variant=2, fused=0),
    "logreg_grad": dict(kind="logreg", n=63, m=2000, d=4096, variant=2, gamma=0.01),
    # wider models at the same 2 GB of samples: 512 threads per CTA (d = 8192), clusters of 4 and 8 CTAs of 4096 columns
    "logreg_grad_d8192": dict(kind="logreg", n=32, m=2000, d=8192, variant=2, gamma=0.01),
    "logreg_grad_d16384": dict(kind="logreg", n=16, m=2000, d=16384, variant=2, gamma=0.01),
    # what ONE of two column shards does per iteration (its half of the columns as a dense block): partial inner
    # products, the sum over shards (here: of its own part alone, in place of the all-reduce), coefficients + A^T pass
    "logreg_grad_shard": dict(kind="shard", n=63, m=2000, d=4096, variant=2, gamma=0.01, shards=2),
    "logreg_grad_d32768": dict(kind="logreg", n=8, m=2000, d=32768, variant=2, gamma=0.01),
    # wider than a cluster of eight holds: the two-pass form (A read twice; the bytes counted are still one pass)
    "logreg_grad_d131072": dict(kind="logreg", n=2, m=2000, d=131072, variant=2, gamma=0.01),
    # whole iterations (gradient kernel + fused step), one CECA cycle captured in a CUDA graph and replayed
    "logreg_train": dict(kind="train", n=63, m=2000, d=4096, variant=2, gamma=0.01, loss="logistic"),
    # the same with a global average (tau + 1 fused consensus rounds) after every second cycle, all inside the graph
    "logreg_train_avg": dict(kind="train", n=63, m=2000, d=4096, variant=2, gamma=0.01, loss="logistic", avg_period=2),
    "logreg_train_small": dict(kind="train", n=5, m=100, d=32, variant=2, gamma=0.05, loss="logistic"),
    "lsq_train": dict(kind="train", n=258, m=50, d=10, variant=1, gamma=0.02, loss="square"),
    # n = 2..128 at d = 4,194,304, both variants where defined: kernel and schedule scaling with n
    "n_sweep": dict(kind="sweep", n=128, d=4_194_304, variant=2, gamma=0.1),
}

FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, each from one ncu
# capture: (bytes per launch, summary under profiles/, source file of the kernel, sha256 prefix of that
# file when the counters were taken).  A kernel source that has changed since makes the entry stale
# and `traffic` is reported as null until the capture is redone.
NCU_TRAFFIC = {
    # 19.73 B per agent-parameter measured on step_small (2.5166 GB read + 1.6220 GB written for
    # 100 x 2,097,152 units); traffic is proportional to the units, scaled to n*d of resnet50_step
    "step_small": (4.1386e9, "dram_traffic__step_consensus_gradient.md", "step.cu", "ceefd77ff7b3"),
    "resnet50_step": (19.734 * 100 * 25_557_032, "dram_traffic__step_consensus_gradient.md", "step.cu", "ceefd77ff7b3"),
    # cycles of two rows (every CECA-1P round): 19.72 B per agent-parameter on step_small's round 6, scaled by units
    "resnet18_step": (19.72 * 24 * 11_689_512, "dram_traffic__step_consensus_gradient.md", "step.cu", "ceefd77ff7b3"),
    # seven launches of a cycle: round 0 moves 1.168 GB, the six others 1.565 GB each
    "consensus_rounds": (10.558e9, "dram_traffic__step_consensus_gradient.md", "step.cu", "ceefd77ff7b3"),
    # fused kernel 2.0735 GB + fixed-order reduce 0.0299 GB
    "logreg_grad": (2.1034e9, "dram_traffic__step_consensus_gradient.md", "logreg.cu", "d1d376d66040"),
    "logreg_grad_d32768": (2.1357e9, "dram_traffic__step_consensus_gradient.md", "logreg.cu", "d1d376d66040"),
    # register-block kernel: captured at d = 2^19 (0.5522 GB per launch) and doubled for d = 2^20 (traffic is per tile)
    "consensus_fused_small": (0.5522e9, "consensus_block_kernel__n97_n258_n1026__ncu_full.md", "consensus_block.cuh", "e5489aec83a7"),
    "consensus_fused": (1.1044e9, "consensus_block_kernel__n97_n258_n1026__ncu_full.md", "consensus_block.cuh", "e5489aec83a7"),
    "consensus_fused_258": (1.5641e9, "consensus_block_kernel__n97_n258_n1026__ncu_full.md", "consensus_block.cuh", "e5489aec83a7"),
    "consensus_fused_1026": (3.1769e9, "consensus_block_kernel__n97_n258_n1026__ncu_full.md", "consensus_block.cuh", "e5489aec83a7"),
    # three-metric captures (dram bytes) of the n = 130 and the 1-port workloads
    "consensus_fused_130": (1.5748e9, "consensus_block_kernel__n97_n258_n1026__ncu_full.md", "consensus_block.cuh", "e5489aec83a7"),
    "consensus_fused_1p": (1.1976e9, "consensus_block_kernel__n97_n258_n1026__ncu_full.md", "consensus_block.cuh", "e5489aec83a7"),
}


def ncu_traffic(workload):
    """Bytes per launch from the recorded capture, or None when there is none or the kernel has changed."""
    import hashlib
    entry = NCU_TRAFFIC.get(workload)
    if entry is None:
        return None
    value, _summary, source, digest = entry
    path = os.path.join(ROOT, "paper_2306_00256_b200", "csrc", source)
    try:
        with open(path, "rb") as f:
            current = hashlib.sha256(f.read()).hexdigest()
    except OSError:
        return None
    return value if current.startswith(digest) else None


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.thread = [], None, None
        self.cmd = ["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                    "-lms", "100"]

    def start(self):
        try:
            self.proc = subprocess.Popen(self.cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [nm for j, nm in enumerate(names) if any(len(r) >= 6 and r[2 + j].lower() == "active" for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def dist_setup(n_gpus):
    """(rank, world, local_rank, dist or None).  Under torchrun the ranks meet over NCCL (gloo without GPUs)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world == 1:
        return 0, 1, 0, None
    import torch
    import torch.distributed as dist
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    backend = "nccl" if torch.cuda.is_available() else "gloo"
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if backend == "nccl":
        torch.cuda.set_device(local_rank)
    dist.init_process_group(backend=backend)
    return dist.get_rank(), world, local_rank, dist


def max_over_ranks(ms, dist, device):
    """The slowest rank's time (device timing, max over ranks)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


# ------------------------------------------------------------------------------------------------
# the oracle on the host cores (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_step_throughput(n, variant, gamma, cols, steps, threads=None):
    import numpy as np
    import oracle
    import synthetic_inputs as synth
    threads = threads or len(os.sched_getaffinity(0))
    oracle.set_threads(threads)
    x, y, g = synth.step_inputs(n, cols, seed=0, x_std=0.01, g_std=0.01)
    x, y, g = x.numpy().astype(np.float64), y.numpy().astype(np.float64), g.numpy().astype(np.float64)
    oracle.step(x, y, g, gamma, variant, 0)  # untimed: loads the library, touches the pages
    t0 = time.perf_counter()
    for k in range(steps):
        x, y = oracle.step(x, y, g, gamma, variant, k)
    dt = time.perf_counter() - t0
    return n * cols * steps / dt, dt / steps, threads


def host_memory_available():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                return int(line.split()[1]) * 1024
    except OSError:
        pass
    return None


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def run_reference(args, wl, rank, world):
    """--impl reference: the fp64 oracle, as it stands, on the host cores, on a column slice."""
    if rank != 0:
        return
    cols = min(wl["d"], 262_144)
    per_step = []
    for _ in range(args.warmup):
        oracle_step_throughput(wl["n"], wl["variant"], wl["gamma"], cols, 1)
    value, sec_per_step, threads = oracle_step_throughput(wl["n"], wl["variant"], wl["gamma"], cols, args.steps)
    sample = "%d-column slice of the %d columns, all %d rows, %d steps; columns are independent, cost is linear in d" % (
        cols, wl["d"], wl["n"], args.steps)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec_per_step * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "n_agents": wl["n"], "d": wl["d"], "variant": "2P" if wl["variant"] == 2 else "1P",
                       "sample_columns": cols},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                             "host_cores": os.cpu_count(), "cpu_model": cpu_model()},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# GPU legs
# ------------------------------------------------------------------------------------------------

def algorithmic_bytes_step(n, d, reads_y):
    """x, e (and y unless its weight is zero) read once; x+, y+ written once; 4 bytes each."""
    return (20 if reads_y else 16) * n * d


def bench_step(args, wl, device, dist):
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth

    n, d, variant, gamma = wl["n"], wl["d"], wl["variant"], wl["gamma"]
    ld = wl.get("ld") or synth.padded_ld(d)  # rows 128-byte aligned: a warp's 512-byte access then covers exactly four lines
    off = int(wl.get("base_offset", 0))
    if off:
        ld = synth.padded_ld(d + off)
        X, Y, G = (torch.as_strided(t, (n, d), (ld, 1), storage_offset=off) for t in
                   synth.step_inputs(n, d + off, seed=0, x_std=0.01, g_std=0.01, device=device, ld=ld))
    else:
        X, Y, G = synth.step_inputs(n, d, seed=0, x_std=0.01, g_std=0.01, device=device, ld=ld)
    storage = wl.get("storage", "f32")
    if storage != "f32":   # the same draws, stored narrow (row by row: no second full-size temporary)
        def narrow(t):
            out = torch.empty((n, ld), dtype=torch.bfloat16, device=device)[:, :d]
            for i in range(n):
                out[i].copy_(t[i])
            return out
        G = narrow(G)
        if storage == "bf16":
            X, Y = narrow(X), narrow(Y)
        torch.cuda.empty_cache()
    bytes_reads_y, bytes_round0 = {"f32": (20, 16), "g_bf16": (18, 14), "bf16": (10, 8)}[storage]
    stream = torch.cuda.current_stream()
    tau = ceca.ceca_schedule(n, variant, 0, peers=False)[0].tau
    x_only = bool(wl.get("x_only"))
    if x_only:
        Y = None
    drop = bool(wl.get("drop_dead_y"))

    def step(k):
        if storage == "f32":
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k, drop_y=drop and k % tau == tau - 1)
        else:
            ceca.ceca_gossip_sgd_step_bf16(X, Y, G, gamma, variant, k)

    k = 0
    for _ in range(args.warmup):
        step(k)
        k += 1
    events = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    k_first = k
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    events[0].record(stream)
    for s in range(args.steps):
        step(k)
        k += 1
        events[s + 1].record(stream)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    clocks = sampler.stop()
    total_ms = events[0].elapsed_time(events[-1])
    per_launch = [events[s].elapsed_time(events[s + 1]) for s in range(args.steps)]
    # dominant kernel: the launches that read Y (every round but r = 0), 20 B per agent-parameter
    dominant = [per_launch[s] for s in range(args.steps)
                if not (drop and (k_first + s) % tau == tau - 1)
                and (x_only or ceca.ceca_schedule(n, variant, k_first + s, peers=False)[0].b_num != 0
                     or ceca.ceca_schedule(n, variant, k_first + s, peers=False)[0].payload == 1)]
    launches = args.steps * ((1 if d % 4 == 0 else 2) + (1 if off else 0))
    roof = None
    if dominant:
        avg_ms = sum(dominant) / len(dominant)
        peak, which = measured_peak()
        achieved = (12 if x_only else bytes_reads_y) * n * d / (avg_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": ncu_traffic(args.workload),
                "kernel": "step_walk_kernel<%s, gradient, %s>" % (
                    {"f32": "float4", "g_bf16": "float4, G bf16", "bf16": "8 columns, X Y G bf16"}[storage],
                    "X only" if x_only else "reads Y"), "peak_source": "of " + which,
                "bytes_per_agent_param": 12 if x_only else bytes_reads_y,
                "avg_launch_ms": avg_ms, "median_launch_ms": statistics.median(dominant), "best_launch_ms": min(dominant),
                "launches_timed": len(dominant),
                "frac_of_nominal_8TBs": achieved / 8000.0,
                "ms_by_round": [round(statistics.mean(per_launch[s] for s in range(args.steps) if (k_first + s) % tau == r), 4)
                                if any((k_first + s) % tau == r for s in range(args.steps)) else None for r in range(tau)]}
    del X, Y, G
    torch.cuda.empty_cache()
    return total_ms, launches, roof, clocks, {"tau": tau, "in_place": True, "ld": ld, "storage": storage,
                                               "l2": "inputs (3 arrays of n x d) far larger than L2"}


def bench_step_e2e(args, wl, device):
    """The same iteration through ceca_gossip_sgd_step_host: pinned host X, Y, G; copies timed."""
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth
    n, d, variant, gamma = wl["n"], wl["d"], wl["variant"], wl["gamma"]
    try:
        hx = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
        hy = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
        hg = torch.empty((n, d), dtype=torch.float32, pin_memory=True)
        pinned = True
    except RuntimeError:
        hx, hy, hg = (torch.empty((n, d), dtype=torch.float32) for _ in range(3))
        pinned = False
    # fill the host buffers from the device generator, one row at a time
    row = torch.empty(d, dtype=torch.float32, device=device)
    gen = torch.Generator(device=device)
    gen.manual_seed(0)
    for i in range(n):
        hx[i].copy_(row.normal_(std=0.01, generator=gen))
    hy.copy_(hx)
    for i in range(n):
        hg[i].copy_(row.normal_(std=0.01, generator=gen))
    del row
    ws = torch.empty(3 << 30, dtype=torch.uint8, device=device)
    steps = max(1, min(args.steps, args.e2e_steps))
    k = 0
    for _ in range(1):
        ceca.ceca_gossip_sgd_step_host(hx, hy, hg, gamma, variant, k, ws)
        k += 1
    h2d = d2h = 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(steps):
        rd = ceca.ceca_schedule(n, variant, k, peers=False)[0]
        reads_y = rd.b_num != 0 or rd.payload == 1
        ceca.ceca_gossip_sgd_step_host(hx, hy, hg, gamma, variant, k, ws)
        h2d += (3 if reads_y else 2) * n * d * 4
        d2h += 2 * n * d * 4
        k += 1
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    return {"value": n * d * steps / dt, "unit": UNIT, "h2d_bytes_per_step": h2d // steps, "d2h_bytes_per_step": d2h // steps,
            "steps": steps, "ms_per_step": dt / steps * 1e3, "pinned": pinned,
            "api": "ceca_gossip_sgd_step_host (column slabs streamed through a 3 GiB device workspace)"}


def bench_consensus(args, wl, device, dist):
    """tau aligned rounds per step (one fused launch, or tau per-round launches); every step has its own
    CUDA-event pair, and the host time of the call (argument checks, schedule, launch) is taken beside it."""
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth
    n, d, variant, fused = wl["n"], wl["d"], wl["variant"], wl["fused"]
    X = synth.consensus_inputs(n, d, seed=1, device=device)
    Xo, Yo = torch.empty_like(X), torch.empty_like(X)
    ws = torch.zeros(64, dtype=torch.int32, device=device)
    tau = ceca.ceca_schedule(n, variant, 0, peers=False)[0].tau
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        ceca.ceca_consensus_rounds(X, None, variant, 0, tau, fused, X_out=Xo, Y_out=Yo, workspace=ws)
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    host_us = []
    torch.cuda.synchronize()
    ev[0].record(stream)
    for s in range(args.steps):
        t0 = time.perf_counter()
        ceca.ceca_consensus_rounds(X, None, variant, 0, tau, fused, X_out=Xo, Y_out=Yo, workspace=ws)
        host_us.append((time.perf_counter() - t0) * 1e6)
        ev[s + 1].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = ev[0].elapsed_time(ev[-1])
    per_call = [ev[s].elapsed_time(ev[s + 1]) for s in range(args.steps)]
    assert ceca.ceca_read_status(ws) == 0
    peak, which = measured_peak()
    per_elem = 12 if fused else (16 * tau - 4)   # fused: X in, X and Y out; per round: 16 B (12 B in round 0)
    avg_ms = total_ms / args.steps
    achieved = per_elem * n * d / (avg_ms * 1e-3) / 1e9
    if not fused:
        kernel = "step_walk_kernel<float4, no gradient> x tau"
    elif fused == 3:
        kernel = "consensus_tmem_kernel (tensor-memory exchange)"
    elif fused == 2 or n > (1152 if variant == 2 else 416):
        kernel = "consensus_fused_kernel (shared-memory exchange of every row)"
    else:
        kernel = "consensus_block_kernel (register blocks, boundary rows through shared memory)"
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": ncu_traffic(args.workload), "kernel": kernel, "peak_source": "of " + which,
            "avg_launch_ms": avg_ms, "median_launch_ms": statistics.median(per_call), "best_launch_ms": min(per_call),
            "host_us_per_call": round(statistics.median(host_us), 1)}
    launches = args.steps * (1 if fused else tau)
    return total_ms, launches, roof, clocks, {"tau": tau, "rounds_per_step": tau,
                                               "l2": "X is %d MB, larger than L2; outputs go to separate buffers" % (n * d * 4 // 1000000)}


def bench_logreg(args, wl, device, dist):
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth
    n, m, d, variant, gamma = wl["n"], wl["m"], wl["d"], wl["variant"], wl["gamma"]
    A, L, _ = synth.logreg_problem(n, m, d, seed=3, flip=0.05, hetero_std=0.5, device=device)
    X = torch.zeros(n, d, device=device); Y = torch.zeros(n, d, device=device); G = torch.empty(n, d, device=device)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=device)
    stream = torch.cuda.current_stream()
    k = 0
    for _ in range(args.warmup):
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        k += 1
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * args.steps + 1)]
    torch.cuda.synchronize()
    ev[0].record(stream)
    for s in range(args.steps):
        ceca.dsgd_logreg_grad(A, L, X, Y, k, variant, G, ws)
        ev[2 * s + 1].record(stream)
        ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)
        ev[2 * s + 2].record(stream)
        k += 1
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = ev[0].elapsed_time(ev[-1])
    grad_ms = sum(ev[2 * s].elapsed_time(ev[2 * s + 1]) for s in range(args.steps)) / args.steps
    peak, which = measured_peak()
    achieved = (4 * n * m * d + 8 * n * d + 4 * n * m) / (grad_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": ncu_traffic(args.workload),
            "kernel": "logreg_fused_kernel + logreg_reduce_kernel", "peak_source": "of " + which, "avg_launch_ms": grad_ms}
    return total_ms, 3 * args.steps, roof, clocks, {"m": m, "l2": "A is %.2f GB, larger than L2" % (4e-9 * n * m * d)}


def bench_shard(args, wl, device, dist):
    """One column shard's share of a column-sharded gradient: A's block is read twice (dots, then A^T coef)."""
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth
    n, m, d, shards = wl["n"], wl["m"], wl["d"], wl["shards"]
    A, L, _ = synth.logreg_problem(n, m, d, seed=3, flip=0.05, hetero_std=0.5, device=device)
    lo, hi = ceca.shard_columns(d, shards, 0)
    As = A[:, :, lo:hi].contiguous()
    del A
    Zs = torch.zeros(n, hi - lo, device=device); Gs = torch.empty(n, hi - lo, device=device)
    total, part = torch.empty(n, m, device=device), torch.empty(n, m, device=device)
    stream = torch.cuda.current_stream()

    def call():
        ceca.dsgd_grad_shard_dots(As, Zs, part)
        ceca.dsgd_grad_shard_sum(total, part, first=True)
        ceca.dsgd_grad_shard_apply(As, L, total, Gs)

    for _ in range(args.warmup):
        call()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(args.steps):
        call()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    peak, which = measured_peak()
    w = hi - lo
    algorithmic = 2 * 4 * n * m * w + 16 * n * m + 8 * n * w     # the block twice, the dots and coefficients, z and G
    achieved = algorithmic / (total_ms / args.steps * 1e-3) / 1e9
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "traffic": None,
            "kernel": "shard_dots_kernel + shard_coef_kernel + shard_accum_vec_kernel", "peak_source": "of " + which,
            "avg_launch_ms": total_ms / args.steps}
    return total_ms, 4 * args.steps, roof, clocks, {"m": m, "shard_columns": [lo, hi], "units": n * w * args.steps,
                                                    "l2": "the shard's block of A is %.2f GB, larger than L2" % (4e-9 * n * m * w)}


def bench_train(args, wl, device, dist):
    """args.steps CECA cycles of (gradient + fused step): eager launches, then one captured cycle replayed."""
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth
    n, m, d, variant, gamma = wl["n"], wl["m"], wl["d"], wl["variant"], wl["gamma"]
    if wl["loss"] == "logistic":
        A, T, _ = synth.logreg_problem(n, m, d, seed=3, flip=0.05, hetero_std=0.5, device=device)
        grad = lambda X, Y, G, k: ceca.dsgd_logreg_grad(A, T, X, Y, k, variant, G, ws)
    else:
        A, T, _ = synth.lsq_problem(n, m, d, seed=0, sigma_s=0.1, device=device)
        noise = synth.gradient_noise(n, d, 0, sigma_n=5.0, device=device)
        grad = lambda X, Y, G, k: ceca.dsgd_lsq_grad(A, T, X, Y, k, variant, G, ws, noise=noise)
    ws = torch.empty(ceca.ceca_workspace_bytes(ceca.WS_LOGREG_GRAD, n, m, d), dtype=torch.uint8, device=device)
    X = torch.zeros(n, d, device=device); Y = torch.zeros(n, d, device=device); G = torch.empty(n, d, device=device)
    tau = ceca.ceca_schedule(n, variant, 0, peers=False)[0].tau

    period = int(wl.get("avg_period", 0))   # cycles between global averages (0: none)
    status = torch.zeros(64, dtype=torch.int32, device=device)

    def one_cycle(k0):
        for k in range(k0, k0 + tau):
            grad(X, Y, G, k)
            ceca.ceca_gossip_sgd_step(X, Y, G, gamma, variant, k)

    def cycle(k0):
        """What one graph replay holds: a CECA cycle, or `period` cycles and a global average."""
        if not period:
            return one_cycle(k0)
        for c in range(period):
            one_cycle(k0 + c * tau)
        ceca.ceca_consensus_rounds(X, Y, variant, k0 + period * tau, tau + 1, 1, workspace=status)

    stream = torch.cuda.current_stream()
    e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
    for c in range(args.warmup):
        cycle(c * tau)
    torch.cuda.synchronize()
    e[0].record(stream)
    for c in range(args.steps):
        cycle(c * tau)
    e[1].record(stream)
    torch.cuda.synchronize()
    eager_ms = e[0].elapsed_time(e[1])
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        cycle(0)
    for _ in range(args.warmup):
        graph.replay()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    stream = torch.cuda.current_stream()
    torch.cuda.synchronize()
    e[2].record(stream)
    for c in range(args.steps):
        graph.replay()
    e[3].record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    graph_ms = e[2].elapsed_time(e[3])
    iters = args.steps * tau * max(period, 1)
    peak, which = measured_peak()
    bytes_per_iter = 4 * n * m * d + 8 * n * d + 4 * n * m + (20 * tau - 4) / tau * n * d
    if period:
        bytes_per_iter += 16 * n * d / (period * tau)   # the fused average: X, Y in and out
    achieved = bytes_per_iter * iters / (graph_ms * 1e-3) / 1e9
    roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "traffic": None,
            "kernel": "gradient kernels + step_walk_kernel, whole iteration", "peak_source": "of " + which,
            "note": "launch-latency bound when n*m*d is small"}
    extra = {"tau": tau, "m": m, "loss": wl["loss"], "iterations_timed": iters, "units": n * d * iters,
             "eager_us_per_iteration": round(eager_ms / iters * 1e3, 2), "graph_us_per_iteration": round(graph_ms / iters * 1e3, 2),
             "l2": "A is %.1f MB" % (n * m * d * 4 / 1e6)}
    launches = iters * 3 + (args.steps if period else 0)
    if period:
        extra["average_every_cycles"] = period
        assert ceca.ceca_read_status(status) == 0
    return graph_ms, launches, roof, clocks, extra


def bench_sweep(args, wl, device, dist):
    """One full CECA cycle (tau fused steps, in place) per n and variant; also the host schedule call."""
    import torch
    import paper_2306_00256_b200 as ceca
    import synthetic_inputs as synth
    n_max, d, gamma = wl["n"], wl["d"], wl["gamma"]
    X, Y, G = synth.step_inputs(n_max, d, seed=0, x_std=0.01, g_std=0.01, device=device)
    stream = torch.cuda.current_stream()
    peak, which = measured_peak()
    rows, launches, total_ms, total_units = [], 0, 0.0, 0
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    for n in range(2, n_max + 1):
        for variant in (2, 1):
            if variant == 1 and n % 2:
                continue
            tau = ceca.ceca_schedule(n, variant, 0, peers=False)[0].tau
            t0 = time.perf_counter()
            for k in range(tau):
                ceca.ceca_schedule(n, variant, k)
            sched_us = (time.perf_counter() - t0) / tau * 1e6
            x, y, g = X[:n], Y[:n], G[:n]
            for k in range(tau):  # warm-up cycle
                ceca.ceca_gossip_sgd_step(x, y, g, gamma, variant, k)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(stream)
            for rep in range(args.steps):
                for k in range(tau):
                    ceca.ceca_gossip_sgd_step(x, y, g, gamma, variant, k)
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / (args.steps * tau)
            gbs = (20 * tau - 4) / tau * n * d / (ms * 1e-3) / 1e9
            rows.append({"n": n, "variant": "2P" if variant == 2 else "1P", "tau": tau, "ms_per_step": round(ms, 4),
                         "updates_per_s": n * d / (ms * 1e-3), "gbs": round(gbs, 1), "frac": round(gbs / peak, 3),
                         "schedule_us": round(sched_us, 2)})
            launches += args.steps * tau
            total_ms += e0.elapsed_time(e1)
            total_units += args.steps * tau * n * d
    clocks = sampler.stop()
    fr = sorted(r["frac"] for r in rows)
    roof = {"bound": "hbm", "achieved": fr[len(fr) // 2] * peak, "peak": peak, "unit": "GB/s", "frac": fr[len(fr) // 2],
            "traffic": None, "kernel": "step_walk_kernel, median over the sweep", "peak_source": "of " + which,
            "min_frac": fr[0], "max_frac": fr[-1]}
    return total_ms, launches, roof, clocks, {"sweep": rows, "units": total_units,
                                               "l2": "n >= 8 rows of 16.8 MB per array exceed L2; smaller n partly L2-resident"}


SECONDARY = ["consensus_fused", "consensus_rounds", "consensus_fused_130", "consensus_fused_258", "consensus_fused_1026",
             "consensus_fused_1p", "logreg_grad", "resnet18_step"]


def run_secondary(device, steps=20, warmup=5):
    """Short legs of the other configurations, attached to the default line as `secondary`: the fused and the
    per-round consensus at n = 97, the fused consensus at the paper's n = 130, 258 and 1026 and with the 1-port
    pairing at n = 100, the logistic gradient
    at n = 63, m = 2000, d = 4096 and the 1-port step at ResNet-18 size.  Each leg is the same function a
    --workload run of that name calls, with its own inputs, warm-up and CUDA events."""
    import torch
    out = []
    for name in SECONDARY:
        wl = WORKLOADS[name]
        sub = argparse.Namespace(steps=steps, warmup=warmup, workload=name)
        fn = {"step": bench_step, "consensus": bench_consensus, "logreg": bench_logreg}[wl["kind"]]
        try:
            total_ms, launches, roof, clocks, _ = fn(sub, wl, device, None)
        except Exception as exc:   # a leg that fails must not take the headline down with it
            out.append({"workload": name, "error": "%s: %s" % (type(exc).__name__, exc)})
            continue
        ms = total_ms / steps
        out.append({"workload": name, "n_agents": wl["n"], "d": wl["d"], "variant": "2P" if wl["variant"] == 2 else "1P",
                    "steps": steps, "warmup": warmup, "ms_per_step": ms, "updates_per_s": wl["n"] * wl["d"] / (ms * 1e-3),
                    "gpu_launches": launches, "clocks": clocks,
                    "roofline": {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "kernel", "peak_source",
                                                      "avg_launch_ms") if k in roof}})
        torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=70)    # ten cycles of the CECA sequence at n = 100 (tau = 7)
    ap.add_argument("--warmup", type=int, default=7)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet50_step", choices=sorted(WORKLOADS))
    ap.add_argument("--e2e-steps", type=int, default=7)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        if wl["kind"] != "step":
            if rank == 0:
                print(json.dumps({"impl": "reference", "unavailable": "the reference arm times the step workloads only"}))
            return
        run_reference(args, wl, rank, int(os.environ.get("WORLD_SIZE", "1")))
        return

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    rank, world, local_rank, dist = dist_setup(args.gpus)
    torch.cuda.set_device(local_rank)
    device = "cuda:%d" % local_rank
    import paper_2306_00256_b200 as ceca
    ceca.library()

    fn = {"step": bench_step, "consensus": bench_consensus, "logreg": bench_logreg, "sweep": bench_sweep,
          "train": bench_train, "shard": bench_shard}[wl["kind"]]
    total_ms, launches, roof, clocks, extra = fn(args, wl, device, dist)
    total_ms = max_over_ranks(total_ms, dist, device)
    units_per_step = wl["n"] * wl["d"]
    value = world * units_per_step * args.steps / (total_ms * 1e-3)
    if wl["kind"] in ("sweep", "train", "shard"):
        value = world * extra.pop("units") / (total_ms * 1e-3)

    e2e = None
    if wl["kind"] == "step" and not args.no_e2e and not wl.get("x_only") and not wl.get("drop_dead_y") and not wl.get("storage"):
        need = world * 3 * units_per_step * 4          # every rank keeps X, Y, G of its block in host memory
        avail = host_memory_available()
        if avail is not None and need > 0.7 * avail:
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                   "unavailable": "host buffers for %d ranks need %.0f GB, the host has %.0f GB available" % (
                       world, need / 1e9, avail / 1e9)}
        else:
            e2e = bench_step_e2e(args, wl, device)
        if dist is not None and e2e.get("value") is not None:
            ms = max_over_ranks(e2e["ms_per_step"], dist, device)
            e2e["ms_per_step"] = ms
            e2e["value"] = world * units_per_step / (ms * 1e-3)

    cpu = None
    if rank == 0 and world == 1 and wl["kind"] == "step" and not args.no_cpu_baseline and not wl.get("storage"):
        cols = min(wl["d"], 262_144)
        v, sec, threads = oracle_step_throughput(wl["n"], wl["variant"], wl["gamma"], cols, 3 * extra["tau"])
        v1, _, _ = oracle_step_throughput(wl["n"], wl["variant"], wl["gamma"], cols // 4, extra["tau"], threads=1)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "%d-column slice (all %d rows), %d steps = 3 cycles of the CECA sequence, fp64" % (cols, wl["n"], 3 * extra["tau"]),
               "single_thread_value": v1, "host_cores": os.cpu_count(), "cpu_model": cpu_model()}

    secondary = None
    if rank == 0 and world == 1 and args.workload == "resnet50_step" and not args.no_secondary:
        secondary = run_secondary(device)

    if rank == 0:
        config = {"workload": args.workload, "n_agents": wl["n"], "d": wl["d"], "variant": "2P" if wl["variant"] == 2 else "1P"}
        config.update(extra)
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic", "config": config, "clocks": clocks, "gpu_launches": launches,
                "e2e": e2e, "roofline": roof, "cpu_baseline": cpu}
        if secondary is not None:
            line["secondary"] = secondary
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
