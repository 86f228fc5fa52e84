"""Embedding-dimension / TT-rank / batch-size sweep of the TT-embedding gather on one GPU.

    python -m paper_2609_03459_b200.sweep [--dims 16,32,64] [--ranks 8,16,32] [--batches 1024,...,131072]
                                          [--train] [--steps 10] [--out table.md]

The axes follow the paper's sensitivity study (Sec. 4.1, embedding dimension d in {16,32,64}, TT-rank in
{8,16,32}, throughput against batch size) plus the paper's own operating point (d=32, rank 32, 3 cores).
Inputs come from `workloads.sweep_point`: 8 tables of the multi-table recipe, the same tables at every
point.  Every timed iteration is bracketed by CUDA events on the launching stream; an L2-sized buffer is
overwritten between iterations because the small-batch points fit the 126 MB L2.  One JSON line per point
on stdout; `--out` also writes a markdown table.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def time_point(D: int, rank: int, batch: int, train: bool, steps: int, warmup: int, device, flush):
    import torch
    import workloads
    from paper_2609_03459_b200 import binding

    wl = workloads.sweep_point(D, rank, batch, with_grad=train)
    emb = binding.from_workload(wl, enable_backward=train, device=device)
    d_idx = torch.from_numpy(wl.indices).to(device)
    d_off = torch.from_numpy(wl.offsets).to(device)
    d_grad = torch.from_numpy(wl.grad_out).to(device) if train else None
    d_out = torch.empty((wl.B, wl.T * wl.D), dtype=torch.float32, device=device)

    def fwd():
        emb.forward(d_idx, d_off, wl.B, out=d_out)

    def step():
        fwd()
        if train:
            emb.backward_sgd(d_grad, wl.lr)

    def timed(fn):
        ms = []
        for i in range(warmup + steps):
            flush.fill_(float(i))          # evict the previous iteration's data from L2
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            if i >= warmup:
                ms.append(e0.elapsed_time(e1))
        return float(np.mean(ms)), float(np.median(ms))

    fwd_mean, fwd_med = timed(fwd)
    counts = emb.grouping_counts()         # of the forward that just ran
    res = {"D": D, "rank": rank, "batch": batch, "tables": wl.T, "lookups": int(wl.L),
           "forward_ms": fwd_mean, "forward_ms_median": fwd_med,
           "forward_lookups_per_s": wl.L / (fwd_mean * 1e-3),
           "distinct_rows": int(counts[:, -1].sum()), "prefix_groups": int(counts[:, -2].sum())}
    if train:
        st_mean, st_med = timed(step)
        res.update({"step_ms": st_mean, "step_ms_median": st_med, "step_lookups_per_s": wl.L / (st_mean * 1e-3)})
    status = emb.status()
    if status != 0:
        raise RuntimeError(f"device status {status} at D={D} rank={rank} batch={batch}")
    del emb
    return res


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--dims", default="16,32,64")
    ap.add_argument("--ranks", default="8,16,32")
    ap.add_argument("--batches", default="1024,4096,16384,32768,131072")
    ap.add_argument("--train", action="store_true", help="also time forward + backward + SGD")
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--out", default="")
    args = ap.parse_args(argv)

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device (there is no CPU fallback)")
    device = torch.device("cuda", 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device).view(torch.float32)

    rows = []
    for D in [int(x) for x in args.dims.split(",")]:
        for rank in [int(x) for x in args.ranks.split(",")]:
            for batch in [int(x) for x in args.batches.split(",")]:
                r = time_point(D, rank, batch, args.train, args.steps, args.warmup, device, flush)
                rows.append(r)
                print(json.dumps(r), flush=True)
    if args.out:
        with open(args.out, "w") as f:
            head = ["D", "rank", "batch", "lookups", "distinct rows", "prefix groups", "forward ms", "forward G lookups/s"]
            if args.train:
                head += ["step ms", "step G lookups/s"]
            f.write("| " + " | ".join(head) + " |\n|" + "---|" * len(head) + "\n")
            for r in rows:
                cells = [r["D"], r["rank"], r["batch"], f"{r['lookups']:,}", f"{r['distinct_rows']:,}",
                         f"{r['prefix_groups']:,}", f"{r['forward_ms']:.3f}", f"{r['forward_lookups_per_s'] / 1e9:.3f}"]
                if args.train:
                    cells += [f"{r['step_ms']:.3f}", f"{r['step_lookups_per_s'] / 1e9:.3f}"]
                f.write("| " + " | ".join(str(c) for c in cells) + " |\n")


if __name__ == "__main__":
    main()
