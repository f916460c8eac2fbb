"""Per-kernel timing of the stand-alone operators, for tuning and for profiler captures.

    python -m paper_2505_16162_b200.opbench linear --n-out 131072 --n-in 5120 --rows 5 --iters 20

times ``knnssd_linear`` on seeded bf16 weights with CUDA events and prints GB/s (weight bytes / time).
Several copies of the matrix are cycled through so that every launch reads from HBM, not from L2.
"""
from __future__ import annotations

import argparse
import json

import torch

import synthetic_inputs as si
from . import build


def bench_linear(n_out: int, n_in: int, rows: int, iters: int, warmup: int, dtype: str = "bf16", pool_gb: float = 2.0):
    build.build()
    from . import binding as kb
    torch.cuda.set_device(0)
    esz = 2 if dtype == "bf16" else 4
    nbytes = n_out * n_in * esz
    copies = max(1, min(16, int(pool_gb * (1 << 30)) // nbytes))
    Ws = [si.normal_weight(7, 100 + i, n_out, n_in, 0.02, dtype, device="cuda") for i in range(copies)]
    x = si.normal_f32(8, 99, torch.arange(rows * n_in, device="cuda"), 1.0).view(rows, n_in).contiguous()
    for i in range(warmup):
        kb.knnssd_linear(Ws[i % copies], x)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        kb.knnssd_linear(Ws[i % copies], x)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / iters
    return {"op": "linear", "n_out": n_out, "n_in": n_in, "rows": rows, "dtype": dtype, "us_per_launch": us,
            "weight_bytes": nbytes, "gbs": nbytes / us / 1e3, "copies_cycled": copies}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["linear"])
    ap.add_argument("--n-out", type=int, default=131072)
    ap.add_argument("--n-in", type=int, default=5120)
    ap.add_argument("--rows", type=int, default=1)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp32"])
    a = ap.parse_args()
    print(json.dumps(bench_linear(a.n_out, a.n_in, a.rows, a.iters, a.warmup, a.dtype)))


if __name__ == "__main__":
    main()
