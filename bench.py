#!/usr/bin/env python
"""Benchmark of the TT-embedding path: pooled lookups/s on seeded synthetic workloads, with roofline.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg3|cfg2|cfg4|cfg1] [--impl reference]

A step is one pass of the whole hot path over one batch: grouping, schedule, contraction, pooling and --
for the training workload (cfg5, the default: the 60-table configuration with backward and SGD) --
the backward pass and the SGD update.  Prints ONE JSON line on rank 0.

  value      lookups/s of the whole job (all ranks), inputs resident in HBM before the timed region
  e2e        the same through the public call with HOST (pinned) buffers: every step uploads one batch
             (indices, offsets, grad_out) and downloads `out` inside the timed region; the upload of step i+1
             overlaps the compute of step i (double-buffered device inputs, copy streams)
  roofline   the dominant kernel of the step against its own bound (measured peaks)
  step_roofline  the whole step against max(FP32 slots / measured FP32 peak, HBM bytes / measured HBM peak)
  cpu_baseline   the fp64 oracle, as it stands, on a bounded sample of the same workload (rank 0, N = 1)

`--impl reference` times the oracle alone on the host cores (same metric, bounded sample per step).
With N > 1 (torchrun) every rank runs the same configuration on its own seeded batch (weak scaling,
batch-sharded replicas); the training step all-reduces the core gradients (NCCL) before SGD.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "pooled TT-embedding lookups/sec at batch 32768 (fwd, fwd+bwd); % of roofline"
UNIT = "lookups/s"
WORKLOADS = {
    "cfg1": (1, False, "config 1: 1 table 100x100x100, D=64, ranks [1,8,8,1], batch 1024, pooling 1, Zipf 1.05, forward"),
    "cfg2": (2, False, "config 2: 1 table 200x250x200, D=128, ranks [1,32,32,1], batch 32768, pooling 20, Zipf 1.1, forward"),
    "cfg3": (3, False, "config 3: 60 tables N~logU[1e4,4e7], D=64, ranks {16,32}, batch 32768, pooling U[1,100], Zipf U[0.8,1.2], forward"),
    "cfg4": (4, False, "config 4: 1 table 64^4, D=128, ranks [1,64,64,64,1], batch 65536, pooling 8, Zipf 1.2, forward"),
    "cfg5": (5, True, "config 5: config-3 tables and indices, forward + backward (grad_out N(0,1)) + SGD lr 0.01"),
    # a shape outside the register-tiled kernel variants: what a user of the any-shape path gets
    "generic": (0, True, "generic path: 8 tables of the config-3 recipe with dim factors 3x3x5 (D=45), ranks [1,6,4,1], "
                         "batch 32768, pooling U[1,100], forward + backward + SGD"),
    # the operating point of the paper's evaluation (Sec. 4.1) on stand-in inputs
    "many-tables": (6, True, "many tables: 240 tables of the config-3 recipe, D=32 (2x4x4), ranks [1,32,32,1], batch 32768, "
                             "bag lengths U[1,P_t] with P_t logU[1,64] per table, forward + backward + SGD"),
}


def make_workload(cfg_id, mapping, num_tables=None, batch=None, batch_seed=None):
    if cfg_id == 6:
        if batch_seed is not None:
            raise SystemExit("the many-tables workload is a single-GPU measurement")
        return workloads.many_tables_point(batch or 32768, num_tables=num_tables or 240, mapping=mapping)
    if cfg_id == 0:
        if batch_seed is not None:
            raise SystemExit("the generic workload is a single-GPU measurement")
        return workloads.generic_point(batch or 32768, num_tables=num_tables or 8, mapping=mapping)
    return workloads.make(cfg_id, mapping=mapping, num_tables=num_tables, batch=batch, batch_seed=batch_seed)


def dram_traffic_per_unit():
    """DRAM bytes per lookup / per distinct row of the gather and sweep kernels from the tracked ncu summary
    (profiles/dram_traffic_per_unit.txt: `kernel unit bytes` lines plus the shape the capture was taken on)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_per_unit.txt")
    res, shape = {}, {}
    if not os.path.exists(path):
        return res, shape
    for ln in open(path):
        f = ln.split("#")[0].split()
        if len(f) == 3 and f[1] in ("lookup", "row"):
            res[f[0]] = (f[1], float(f[2]))
        elif len(f) == 2 and f[0].startswith("capture_"):
            shape[f[0]] = f[1]
    return res, shape


# ------------------------------------------------------------------------------------------------ helpers

def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (profiling recipe)"


class ClockSampler:
    """nvidia-smi clock / throttle samples while a timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()  # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def sample_bags(wl, stride: int):
    """Every stride-th bag of every table, as a list of per-table (indices, offsets, bag ids)."""
    res = []
    for t in range(wl.T):
        idx, off = wl.table_slice(t)
        bags = np.arange(0, wl.B, stride)
        lens = (off[1:] - off[:-1])[bags]
        sub_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        sub_idx = np.concatenate([idx[off[b]:off[b + 1]] for b in bags]) if len(bags) else np.zeros(0, np.int64)
        res.append((sub_idx, sub_off, bags))
    return res


def oracle_pass(wl, sample, train: bool) -> int:
    """One pass of the fp64 oracle (as it stands) over the sampled bags; returns lookups processed."""
    import oracle
    n = 0
    D = wl.D
    for t, (idx, off, bags) in enumerate(sample):
        s = wl.tables[t]
        oracle.forward(s.n, s.d, s.r, s.N, wl.cores[t], idx, off)
        if train:
            g = oracle.backward(s.n, s.d, s.r, s.N, wl.cores[t], idx, off, wl.grad_out[bags, t * D:(t + 1) * D])
            oracle.sgd(wl.cores[t], g, wl.lr)
        n += idx.shape[0]
    return n


def pick_stride(wl, train: bool) -> int:
    # aim at roughly 10-30 s of CPU work for the sample (measured rates of the plain oracle: ~0.5 M lookups/s
    # forward, ~0.1 M lookups/s with backward, at rank 32 on 8 cores; scaled by the contraction size)
    spec = wl.tables[0]
    K = spec.K
    fma = 0
    P = 1
    for k in range(K):
        fma += P * spec.r[k] * spec.d[k] * spec.r[k + 1]
        P *= spec.d[k]
    per_lookup = fma * (4.0 if train else 1.0)
    budget = 15.0 * 14e9  # the plain oracle sustains ~14 G fp64 FMA/s on the 16 host cores of the GPU machine
    want = max(1.0, budget / per_lookup)
    stride = int(max(1, round(wl.L / want)))
    return min(stride, max(1, wl.B // 4))


# ------------------------------------------------------------------------------------------------ algorithmic work

def algorithmic_work(wl, counts, train: bool):
    """FP32 slots (FMA or ADD lanes) and HBM bytes the method itself needs after de-duplication."""
    T, K, D, L, B = wl.T, wl.tables[0].K, wl.D, wl.L, wl.B
    s_contract = 0
    touched_core_bytes = 0
    seg_adds = 0
    for t, s in enumerate(wl.tables):
        P = 1
        for k in range(1, K + 1):           # level k uses core k (1-based)
            c_k = P * s.r[k - 1] * s.d[k - 1] * s.r[k]
            if k >= 2:
                s_contract += int(counts[t, k - 1]) * c_k
            slice_f = s.r[k - 1] * s.d[k - 1] * s.r[k]
            touched_core_bytes += min(int(counts[t, k - 1]), s.n[k - 1]) * slice_f * 4
            seg_adds += int(counts[t, k - 1]) * slice_f
            P *= s.d[k - 1]
    U = int(counts[:, K - 1].sum())
    core_bytes = sum(c.size * 4 for tc in wl.cores for c in tc)
    # L2 -> SM bytes the design's ordering implies (slice fetches): forward one slice of core K-1 per batch of four
    # groups (digit-major order) and one slice of core K per distinct row; backward one slice of core K-1 per group,
    # the slice of core K once per row pass (two passes), and each dE row twice
    l2_fwd = l2_bwd = 0
    for t, s in enumerate(wl.tables):
        if K >= 3:
            mid_slice = s.r[K - 2] * s.d[K - 2] * s.r[K - 1] * 4
            l2_fwd += int(counts[t, K - 2]) * mid_slice // 4
            l2_bwd += int(counts[t, K - 2]) * mid_slice * 2     # recompute of C and the middle-core backward
        last_slice = s.r[K - 1] * s.d[K - 1] * 4
        l2_fwd += int(counts[t, K - 1]) * last_slice
        l2_bwd += int(counts[t, K - 1]) * (2 * last_slice + 2 * D * 4)
    fwd_slots = s_contract + L * D
    fwd_bytes = 8 * L + 8 * (T * B + 1) + 8 * U + min(touched_core_bytes, core_bytes) + 4 * B * T * D
    res = {"U_rows": U, "U_prefix": int(counts[:, K - 2].sum()), "fwd_slots": fwd_slots, "fwd_hbm_bytes": fwd_bytes,
           "contract_slots": s_contract, "pool_slots": L * D, "fwd_l2_bytes": l2_fwd,
           "pool_kernel_bytes": 8 * L + 8 * (T * B + 1) + 4 * U * D + 4 * B * T * D}
    if train:
        # dE sums; dD and dC per row and the level above (2x the forward contractions), recompute of the
        # on-chip intermediates (levels below K), segment-reduce adds of the slice gradients
        recompute = 0
        for t, s in enumerate(wl.tables):
            P = 1
            for k in range(1, K):
                if k >= 2:
                    recompute += int(counts[t, k - 1]) * P * s.r[k - 1] * s.d[k - 1] * s.r[k]
                P *= s.d[k - 1]
        bwd_slots = L * D + 2 * s_contract + recompute + seg_adds
        bwd_bytes = 8 * L + 4 * B * T * D + core_bytes + 3 * core_bytes
        res.update({"bwd_slots": bwd_slots, "bwd_hbm_bytes": bwd_bytes, "bwd_l2_bytes": l2_bwd,
                    "dE_kernel_bytes": 8 * L + 4 * B * T * D + 4 * U * D})
    return res


# ------------------------------------------------------------------------------------------------ reference arm

def run_reference(args, wl, train, desc, rank, world):
    if rank != 0:
        return
    stride = args.cpu_stride or pick_stride(wl, train)
    sample = sample_bags(wl, stride)
    cores = len(os.sched_getaffinity(0))
    for _ in range(max(args.warmup, 0) and 1):
        oracle_pass(wl, sample, train)
    t0 = time.perf_counter()
    n = 0
    for _ in range(args.steps):
        n += oracle_pass(wl, sample, train)
    dt = time.perf_counter() - t0
    v = n / dt
    sample_desc = f"every {stride}-th bag of every table ({n // args.steps} lookups per step), fp64 oracle, OpenMP over bags"
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": desc, "mapping": args.mapping, "sample": sample_desc},
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample_desc},
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ launcher

def launch_ranks(n: int) -> int:
    """Re-run this command line as n ranks (torch.distributed.run, one process per GPU, rendezvous on 127.0.0.1).
    Fails before starting anything when the node has fewer than n GPUs.  Returns the exit code."""
    import socket
    import torch
    have = torch.cuda.device_count()
    if have < n:
        print(f"bench.py: --gpus {n} needs {n} GPUs on this node, {have} visible; not running on fewer", file=sys.stderr)
        return 2
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.run(cmd).returncode


# ------------------------------------------------------------------------------------------------ main arm

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=sorted(WORKLOADS))
    ap.add_argument("--mapping", default="identity", choices=["identity", "scattered"])
    ap.add_argument("--cpu-stride", type=int, default=0, help="bag stride of the oracle sample (0 = automatic)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--ablation", default="none", choices=["none", "unique-only", "static", "unique-only+static", "no-dedup"],
                    help="study switches (forward workloads only): no prefix reuse / equal-count schedule / no de-duplication")
    ap.add_argument("--num-tables", type=int, default=0, help="reduced case for profiler captures: fewer tables (cfg3/cfg5)")
    ap.add_argument("--batch", type=int, default=0, help="reduced case for profiler captures: smaller batch")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # called plainly with --gpus N: start the N ranks ourselves (one process per GPU) and hand over
        raise SystemExit(launch_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "ours" and world != max(args.gpus, 1):
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}: launch one rank per GPU")
    cfg_id, train, desc = WORKLOADS[args.workload]

    if args.impl == "reference":
        if rank != 0:
            return
        wl = make_workload(cfg_id, args.mapping)
        run_reference(args, wl, train, desc, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_03459_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback); use --impl reference for the oracle")
    if torch.cuda.device_count() < world or local_rank >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: {world} ranks asked for, {torch.cuda.device_count()} GPUs visible "
                         "(one rank per GPU; nothing is run on fewer)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        # communicator set-up lines (rings / trees / NVLS) go to stderr: the JSON line stays alone on stdout
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT,GRAPH")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=device)

    # every rank draws its own batch from the same recipe (weak scaling); tables/cores are identical
    shrink = dict(num_tables=args.num_tables or None, batch=args.batch or None)
    wl = make_workload(cfg_id, args.mapping, **shrink) if rank == 0 else None
    if shrink["num_tables"] or shrink["batch"]:
        desc += f" [REDUCED: tables={shrink['num_tables'] or 'all'}, batch={shrink['batch'] or 'full'}]"
    from paper_2609_03459_b200 import dist as ttd
    if rank > 0:
        wl = make_workload(cfg_id, args.mapping, batch_seed=ttd.rank_seed(workloads.BASE_SEED, rank), **shrink)
    T, K, D, B, L = wl.T, wl.tables[0].K, wl.D, wl.B, wl.L
    L_all = ttd.sum_over_ranks(L, device=device) if world > 1 else L   # lookups of the whole job (every rank has its own batch)

    abl = {"none": 0, "unique-only": 1, "static": 2, "unique-only+static": 3, "no-dedup": 4}[args.ablation]
    if abl and train:
        raise SystemExit("--ablation needs a forward workload (cfg1..cfg4)")
    # Room for distinct rows: the safe bound min(L, sum N) would size the row buffer for 99 M rows (25 GB) on the 60-table
    # workload, whose batches hold about 0.2 L distinct rows.  Large batches get L / 4 rows; a batch with more would set the
    # overflow status bit, which is checked below.
    # (the many-tables workload, with its short bags, holds 0.25 L: it gets L / 2)
    mur = 0 if (abl & 4) else max(L // (2 if cfg_id == 6 else 4), min(L, 1 << 22))
    emb = binding.from_workload(wl, enable_backward=train, ablation=abl, max_unique_rows=mur, device=device)
    h_idx = torch.from_numpy(wl.indices).pin_memory()
    h_off = torch.from_numpy(wl.offsets).pin_memory()
    h_grad = torch.from_numpy(wl.grad_out).pin_memory() if train else None
    h_out = torch.empty((B, T * D), dtype=torch.float32).pin_memory()
    d_idx, d_off = h_idx.to(device), h_off.to(device)
    d_grad = h_grad.to(device) if train else None
    d_out = torch.empty((B, T * D), dtype=torch.float32, device=device)

    def step(idx, off, grad):
        emb.forward(idx, off, B, out=d_out)
        if train and world == 1:
            emb.backward_sgd(grad, wl.lr)              # the update rides on the kernels that finalise each gradient
        elif train:
            emb.backward(grad)
            ttd.allreduce_core_grads(emb.flat_grads)   # the one exchange of the data-parallel path
            emb.sgd_step(wl.lr)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, after=None):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        if after is not None:
            after()       # e.g. join side streams so that their work falls inside the timed region
        e1.record()
        barrier()
        ms = torch.tensor([e0.elapsed_time(e1)], device=device)
        if world > 1:
            dist.all_reduce(ms, op=dist.ReduceOp.MAX)
        return float(ms.item())

    # ---- roofline denominators measured in this run
    fp32_peak = binding.probe_fp32()
    mma_peak = binding.probe_mma()   # warp-level mma.sync m16n8k8 TF32 instructions per second
    # the same products as tcgen05 instructions (M 128, k 8), for the two output widths the path has: TFLOP/s-equivalent
    tc5 = {}
    for n_cols in (128, 32):
        rate5, err5 = binding.probe_tcgen05(n_cols)
        tc5["n%d_tflops" % n_cols] = rate5 * 2.0 * 128 * n_cols * 8 / 1e12
        tc5["n%d_max_abs_err" % n_cols] = err5
    l2_gather = binding.probe_gather(32 << 20, device=device)
    hbm_gather = binding.probe_gather(2 << 30, device=device)
    hbm_gbs, peak_src = measured_peaks()

    for _ in range(args.warmup):
        step(d_idx, d_off, d_grad)
    torch.cuda.synchronize()
    status = emb.status()
    if status & binding.STATUS_OVERFLOW:
        raise SystemExit("bench.py: more distinct rows than max_unique_rows; the timed work would be incomplete")

    sampler = ClockSampler(local_rank)
    sampler.start()
    # ---- device-resident timing of the whole step, per-stage events enabled
    emb.enable_timing(True)
    stage_tot = {}
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    binding.launch_count(reset=True)
    for _ in range(args.steps):
        step(d_idx, d_off, d_grad)
    launches_per_step = binding.launch_count() / max(args.steps, 1)   # counted at the library's launch sites
    e1.record()
    barrier()
    total_ms = e0.elapsed_time(e1)
    # per-stage averages: events of the last step are still valid; re-run a few steps to average them
    stage_acc = {}
    for _ in range(min(args.steps, 5)):
        step(d_idx, d_off, d_grad)
        torch.cuda.synchronize()
        for k, v in emb.stage_ms().items():
            stage_acc.setdefault(k, []).append(v)
    stage_ms = {k: float(np.mean(v)) for k, v in stage_acc.items()}
    # per-kernel durations of the shape-variant kernels: in the timed region they share the GPU on forked streams, so
    # a few extra steps run them one after the other (timing mode 2) to get each kernel's own duration
    emb.enable_timing(2)
    solo_acc = {}
    for i in range(4):
        step(d_idx, d_off, d_grad)
        torch.cuda.synchronize()
        if i:
            for k, v in emb.stage_ms().items():
                if k.startswith("k_sweep_"):
                    solo_acc.setdefault(k, []).append(v)
    solo_ms = {k: float(np.mean(v)) for k, v in solo_acc.items()}
    emb.enable_timing(False)
    ms_t = torch.tensor([total_ms], device=device)
    if world > 1:
        dist.all_reduce(ms_t, op=dist.ReduceOp.MAX)
    total_ms = float(ms_t.item())
    ms_per_step = total_ms / args.steps

    # ---- forward only (same inputs)
    fwd_ms = timed(lambda: emb.forward(d_idx, d_off, B, out=d_out), args.steps) / args.steps
    # the same forward replayed from a CUDA graph (fixed buffers): what the launch-latency-bound small batches gain
    fwd_graph_ms = None
    if not train and L <= 4_000_000:
        graph = emb.capture_forward(d_idx, d_off, B, d_out)
        for _ in range(3):
            graph.replay()
        fwd_graph_ms = timed(graph.replay, args.steps) / args.steps
        del graph

    # ---- end to end through host buffers
    e2e = None
    if not args.no_e2e:
        # The loop a user runs with host buffers, software-pipelined like a data loader: the inputs of step i+1
        # (indices, offsets, grad_out) go up on a copy stream while step i computes, `out` of step i comes down on a
        # third stream while its backward runs.  Every step uploads one batch and downloads one result inside the
        # timed region; the device buffers are double-buffered, the hazards are ordered with events.
        up, down = torch.cuda.Stream(device), torch.cuda.Stream(device)

        def run_e2e(h_ids):
            """Pipelined loop with the row ids taken from the pinned host tensor h_ids (int64 or int32)."""
            e_idx = [torch.empty(h_ids.shape, dtype=h_ids.dtype, device=device) for _ in range(2)]
            e_off = [torch.empty_like(d_off) for _ in range(2)]
            e_grad = [torch.empty_like(d_grad) for _ in range(2)] if train else None
            e_out = [d_out, torch.empty_like(d_out)]     # double-buffered result: its download overlaps the next forward
            state = {"i": 0, "ready": [None, None], "free": [None, None], "out_done": [None, None]}

            def upload(slot):
                # batch for buffer `slot`: waits until the step that last used the buffer is over
                if state["free"][slot] is not None:
                    up.wait_event(state["free"][slot])
                with torch.cuda.stream(up):
                    e_idx[slot].copy_(h_ids, non_blocking=True)
                    e_off[slot].copy_(h_off, non_blocking=True)
                    if train:
                        e_grad[slot].copy_(h_grad, non_blocking=True)
                    state["ready"][slot] = up.record_event()

            def e2e_step():
                main = torch.cuda.current_stream()
                i = state["i"]
                slot = i & 1
                if state["ready"][slot] is None:
                    upload(slot)                       # first step: nothing was prefetched yet
                main.wait_event(state["ready"][slot])
                if state["out_done"][slot] is not None:
                    main.wait_event(state["out_done"][slot])  # the result of two steps ago has left this buffer
                upload(slot ^ 1)                       # prefetch the next batch while this one computes
                emb.forward(e_idx[slot], e_off[slot], B, out=e_out[slot])
                ev_fwd = main.record_event()
                down.wait_event(ev_fwd)
                with torch.cuda.stream(down):
                    h_out.copy_(e_out[slot], non_blocking=True)
                    state["out_done"][slot] = down.record_event()
                if train and world == 1:
                    emb.backward_sgd(e_grad[slot], wl.lr)
                elif train:
                    emb.backward(e_grad[slot])
                    ttd.allreduce_core_grads(emb.flat_grads)
                    emb.sgd_step(wl.lr)
                state["free"][slot] = main.record_event()
                state["ready"][slot] = None
                state["i"] = i + 1

            def e2e_drain():
                main = torch.cuda.current_stream()
                main.wait_stream(up)
                main.wait_stream(down)
            for _ in range(2):
                e2e_step()
            e2e_drain()
            ms = timed(lambda: e2e_step(), args.steps, after=e2e_drain) / args.steps
            torch.cuda.synchronize()
            return ms

        e2e_ms = run_e2e(h_idx)
        # the same loop with 32-bit row ids (tt_emb_forward_i32): half the index bytes over PCIe
        h_idx32 = h_idx.to(torch.int32).pin_memory()
        e2e32_ms = run_e2e(h_idx32)
        h2d = h_idx.numel() * 8 + h_off.numel() * 8 + (h_grad.numel() * 4 if train else 0)
        e2e = {"value": L_all / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(h_out.numel() * 4),
               "int32_ids": {"value": L_all / (e2e32_ms * 1e-3), "ms_per_step": e2e32_ms,
                             "h2d_bytes_per_step": int(h2d - h_idx.numel() * 4)}}
    clocks = sampler.stop()

    emb.forward(d_idx, d_off, B, out=d_out)
    torch.cuda.synchronize()
    counts = emb.grouping_counts()
    work = algorithmic_work(wl, counts, train)

    # ---- roofline of the dominant kernel and of the whole step
    # DRAM traffic per lookup / per distinct row of the top kernels comes from the tracked ncu summary of a reduced case
    # and is scaled by the units this launch processes; it is reported only for the shape the capture was taken on.
    ncu_traffic, capture = dram_traffic_per_unit()
    pool_kernel = "k_pool_async" if 16 < D <= 64 and D % 4 == 0 else ("k_pool_vec" if D % 4 == 0 else "k_pool_scalar")
    if pool_kernel == "k_pool_async" and L < (12 if D > 32 else 33) * T * B:
        pool_kernel = "k_pool_stream"   # the library's choice for short bags (windows of lookups across bags)
    same_shape = capture.get("capture_D") == str(D) and capture.get("capture_recipe") in ("cfg3", "cfg5") and cfg_id in (3, 5)

    def traffic_of(kernel, share=1.0):
        if not same_shape or kernel not in ncu_traffic:
            return None
        unit, per = ncu_traffic[kernel]
        return per * (wl.L if unit == "lookup" else work["U_rows"] * share)

    # sweep kernel variant of every table, as the library assigned it
    table_variant = [emb.table_variant(t) for t in range(T)]
    variant_rows = {}   # distinct rows handled by each sweep variant
    for t in range(T):
        variant_rows[table_variant[t]] = variant_rows.get(table_variant[t], 0) + int(counts[t, K - 1])

    def variant_slots(v, backward):
        tot = 0
        for t, s in enumerate(wl.tables):
            if table_variant[t] != v:
                continue
            P = int(np.prod(s.d[:K - 2])) if K >= 3 else 1
            c_mid = P * s.r[K - 2] * s.d[K - 2] * s.r[K - 1] if K >= 3 else 0
            c_last = int(np.prod(s.d[:K - 1])) * s.r[K - 1] * s.d[K - 1]
            g, u = int(counts[t, K - 2]), int(counts[t, K - 1])
            tot += (g * c_mid + 2 * u * c_last) if backward else (g * c_mid + u * c_last)
        return tot

    kernels = {}
    if "pooling" in stage_ms:
        ms = stage_ms["pooling"]
        ach = work["pool_kernel_bytes"] / (ms * 1e-3) / 1e9
        kernels[pool_kernel] = (ms, {"kernel": pool_kernel, "bound": "hbm", "achieved": ach, "peak": hbm_gbs, "unit": "GB/s",
                                      "frac": ach / hbm_gbs, "traffic": traffic_of("k_pool"), "peak_source": peak_src,
                                      "note": "algorithmic bytes: indices + offsets + every distinct row once + out "
                                              "(+ one (slot,bag) pair per lookup when the backward is enabled); the "
                                              "per-lookup row gather (L*D*4 bytes) is on-chip / re-read traffic and is "
                                              "not counted; traffic scaled from the reduced-case ncu capture named in "
                                              "profiles/dram_traffic_per_unit.txt (null for other shapes)",
                                      "frac_without_row_buffer": (8 * L + 8 * (T * B + 1) + 4 * B * T * D) / (ms * 1e-3) / 1e9 / hbm_gbs,
                                      "row_gather_GBs": wl.L * D * 4 / (ms * 1e-3) / 1e9,
                                      "row_gather_peak_l2_GBs": l2_gather / 1e9, "row_gather_peak_hbm_GBs": hbm_gather / 1e9})
    if train and "bwd_dE" in stage_ms:
        ms = stage_ms["bwd_dE"]
        ach = work["dE_kernel_bytes"] / (ms * 1e-3) / 1e9
        de_kernel = "k_dE_stage" if D in (16, 32, 64) else "k_dE_fast"
        kernels[de_kernel] = (ms, {"kernel": de_kernel + " (+k_dE_fix)", "bound": "hbm", "achieved": ach, "peak": hbm_gbs,
                                     "unit": "GB/s", "frac": ach / hbm_gbs, "traffic": traffic_of("k_dE"),
                                     "peak_source": peak_src})
    for name, ms in solo_ms.items():
        if name.startswith("k_sweep_"):
            v = int(name[name.index("<") + 1:name.index(">")])
            bwd = name.startswith("k_sweep_bwd")
            slots = variant_slots(v, bwd)
            ach = slots / (ms * 1e-3) / 1e12
            share = variant_rows.get(v, 0) / max(work["U_rows"], 1)
            # the same work in the unit of the tensor path: three m16n8k8 instructions per 1024 slots if every product
            # ran there (the forward sweeps do; the backward sweeps rebuild the intermediate product on the FP32 pipe);
            # padding of the small shape variants is not counted
            mma_min = 3.0 * slots / 1024.0
            kernels[name] = (ms, {"kernel": name, "bound": "alu", "achieved": ach, "peak": fp32_peak / 1e12,
                                  "unit": "T FP32 lane-ops/s", "frac": ach / (fp32_peak / 1e12),
                                  "mma_sync": {"instructions_equiv": mma_min, "per_s": mma_min / (ms * 1e-3), "peak_per_s": mma_peak,
                                               "frac_equiv": mma_min / (ms * 1e-3) / mma_peak},
                                  "traffic": traffic_of("k_sweep_bwd" if bwd else "k_sweep_fwd", share),
                                  "peak_source": "independent-FMA-chain probe in this run",
                                  "note": "FMA-equivalent slots of the contractions this kernel performs; the row stages "
                                          "run as 3xTF32 tensor-core products, the peak is the FP32 pipe; duration from "
                                          "extra steps that run the shape-variant kernels one after the other (in the "
                                          "timed region they overlap on forked streams: see stage_ms)"})
    if kernels:
        dominant = max(kernels, key=lambda k: kernels[k][0])
        roofline = dict(kernels[dominant][1], ms_per_launch=kernels[dominant][0])
    else:
        roofline = None
    kernel_rooflines = {k: dict({"ms": v[0], "frac": v[1]["frac"], "bound": v[1]["bound"]},
                                **({"mma_sync_frac_equiv": v[1]["mma_sync"]["frac_equiv"]} if "mma_sync" in v[1] else {}))
                        for k, v in kernels.items()}
    tot_slots = work["fwd_slots"] + (work["bwd_slots"] if train else 0)
    tot_bytes = work["fwd_hbm_bytes"] + (work["bwd_hbm_bytes"] if train else 0)
    tot_l2 = work["fwd_l2_bytes"] + (work["bwd_l2_bytes"] if train else 0)
    t_alu, t_hbm, t_l2 = tot_slots / fp32_peak, tot_bytes / (hbm_gbs * 1e9), tot_l2 / l2_gather
    t_roof = max(t_alu, t_hbm, t_l2)
    step_roof = {"t_alu_ms": t_alu * 1e3, "t_hbm_ms": t_hbm * 1e3, "t_l2_ms": t_l2 * 1e3,
                 "bound": "alu" if t_roof == t_alu else ("hbm" if t_roof == t_hbm else "l2"),
                 "t_roof_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms_per_step,
                 "fp32_slots": tot_slots, "hbm_bytes": tot_bytes, "l2_bytes": tot_l2,
                 "l2_peak_note": "L2 term against the measured 256-byte-row gather rate from an L2-resident buffer"}
    fwd_roof_t = max(work["fwd_slots"] / fp32_peak, work["fwd_hbm_bytes"] / (hbm_gbs * 1e9), work["fwd_l2_bytes"] / l2_gather)

    line = {
        "metric": METRIC, "value": L_all / (ms_per_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": desc, "mapping": args.mapping, "tables": T, "batch_per_gpu": B, "lookups_per_gpu": L,
                   "step": "forward+backward+sgd" if train else "forward", "ablation": args.ablation,
                   "parallelism": f"dp{world} (batch-sharded replicas" + (", all-reduce of core gradients)" if train else ")"),
                   "l2_policy": "inputs larger than L2 (indices alone are %.0f MB)" % (L * 8 / 1e6)},
        "forward_only": {"value": L_all / (fwd_ms * 1e-3), "unit": UNIT, "ms_per_step": fwd_ms,
                         "roofline_frac": fwd_roof_t * 1e3 / fwd_ms, "t_roof_ms": fwd_roof_t * 1e3,
                         "cuda_graph_ms_per_step": fwd_graph_ms},
        "stage_ms": stage_ms, "solo_kernel_ms": solo_ms, "roofline": roofline, "kernel_rooflines": kernel_rooflines, "step_roofline": step_roof,
        "peaks": {"hbm_GBs": hbm_gbs, "hbm_source": peak_src, "fp32_lane_ops_per_s": fp32_peak,
                  "mma_sync_tf32_m16n8k8_per_s": mma_peak, "mma_sync_tf32_tflops": mma_peak * 2048 / 1e12,
                  "tcgen05_tf32": tc5,
                  "l2_row_gather_GBs": l2_gather / 1e9, "hbm_row_gather_GBs": hbm_gather / 1e9},
        "work": work, "device_status": status, "clocks": clocks, "e2e": e2e,
        "gpu_launches": int(round(launches_per_step)),
        "workspace_GB": emb.workspace_bytes / 1e9,
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        stride = args.cpu_stride or pick_stride(wl, train)
        sample = sample_bags(wl, stride)
        t0 = time.perf_counter()
        n = oracle_pass(wl, sample, train)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": n / dt, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": f"every {stride}-th bag of every table ({n} lookups, {dt:.1f} s), fp64, "
                                          "same step (forward" + ("+backward+sgd)" if train else ")")}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
