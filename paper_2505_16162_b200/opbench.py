"""Per-kernel timing, for tuning and for profiler captures.

    python -m paper_2505_16162_b200.opbench linear --n-out 131072 --n-in 5120 --rows 5 --iters 20

times ``knnssd_linear`` on seeded bf16 weights with CUDA events and prints GB/s (weight bytes / time).
Several copies of the matrix are cycled through so that every launch reads from HBM, not from L2.  ``linear_tc`` with
the same options times the stand-alone tensor-core form (``knnssd_linear_tc``, up to 16 rows).

    python -m paper_2505_16162_b200.opbench pass --shape llama13b --layers 4 --context 1280 --rows 5 --iters 10

times the persistent pass kernel (rows 1 = a draft step under a seeded 45 % skip mask, rows k+1 = a verification pass)
on a model of the named widths cut to ``--layers`` layers, small enough for a multi-pass profiler capture.

    python -m paper_2505_16162_b200.opbench prompt --shape llama13b --layers 4 --context 1024 --iters 5

times the tensor-core prompt pass (``knnssd_prefill``) over ``--context`` rows and prints the tensor-core rate of its
linear maps (both bf16 terms of the activations counted: 4 x rows x weights FLOP).

    python -m paper_2505_16162_b200.opbench anchors --n-out 5 --rows 1000 --n-in 5120 --iters 10

times anchor construction (``knnssd_build_anchors``: ``--n-out`` domains x ``--rows`` sampled vectors of width
``--n-in``, 10 anchors each) from a start inside one domain, and prints the device time per K-means round and the
rate at which a round reads the points (twice per round: assignment and centroid sums).
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


def bench_linear_tc(n_out: int, n_in: int, rows: int, iters: int, warmup: int, pool_gb: float = 2.0):
    """The stand-alone tensor-core linear map (``knnssd_linear_tc``), timed by its own CUDA events."""
    build.build()
    from . import binding as kb
    torch.cuda.set_device(0)
    nbytes = n_out * n_in * 2
    copies = max(1, min(16, int(pool_gb * (1 << 30)) // nbytes))
    Ws = [si.normal_weight(7, 100 + i, n_out, n_in, 0.02, "bf16", device="cuda") for i in range(copies)]
    x = si.normal_f32(8, 99, torch.arange(rows * n_in, device="cuda"), 1.0).view(rows, n_in).contiguous()
    ms = []
    for i in range(warmup + iters):
        _, t = kb.knnssd_linear_tc(Ws[i % copies], x)
        if i >= warmup:
            ms.append(t)
    ms.sort()
    med = ms[len(ms) // 2]
    return {"op": "linear_tc", "n_out": n_out, "n_in": n_in, "rows": rows, "us_per_call": med * 1e3,
            "weight_bytes": nbytes, "gbs": nbytes / med / 1e6, "copies_cycled": copies}


def bench_pass(shape_name: str, layers: int, context: int, rows: int, iters: int, seed: int = 0):
    build.build()
    from . import binding as kb
    import numpy as np
    torch.cuda.set_device(0)
    shape = si.SHAPES[shape_name].with_layers(layers)
    w = si.make_model_weights(shape, seed, device="cuda")
    n_skip = int(round(0.45 * 2 * layers))
    mask = si.skip_mask(seed + 102, 2 * layers, n_skip)
    sess = kb.Session.from_shape(shape, w, context + 64, max_draft=8)
    prompt = si.uniform_tokens(seed, 0, context, shape.vocab).numpy()
    sess.prefill(prompt)
    sess.set_skipmask(mask)
    which, k = (0, 1) if rows == 1 else (1, rows - 1)
    t = sess.time_pass(which, k, iters)
    b = 2 if shape.dtype == "bf16" else 4
    d, hd = shape.d_model, shape.head_dim
    attn_w = (2 * d * shape.n_heads * hd + 2 * d * shape.n_kv_heads * hd) * b
    mlp_w, head_w = 3 * d * shape.d_ff * b, shape.vocab * d * b
    kv = 2 * shape.n_kv_heads * hd * b * (context + rows)
    use = (lambda j: True) if rows > 1 else (lambda j: not mask[j])
    n_attn = sum(1 for l in range(layers) if use(2 * l))
    n_mlp = sum(1 for l in range(layers) if use(2 * l + 1))
    nbytes = n_attn * (attn_w + kv) + n_mlp * mlp_w + head_w
    return {"op": "pass", "shape": shape.name, "rows": rows, "context": context, "ms_per_pass": t["ms_per_pass"],
            "algorithmic_bytes": nbytes, "gbs": nbytes / t["ms_per_pass"] / 1e6,
            "attention_sublayers": n_attn, "mlp_sublayers": n_mlp}


def bench_prompt(shape_name: str, layers: int, rows: int, iters: int, seed: int = 0):
    build.build()
    from . import binding as kb
    torch.cuda.set_device(0)
    shape = si.SHAPES[shape_name].with_layers(layers)
    w = si.make_model_weights(shape, seed, device="cuda")
    sess = kb.Session.from_shape(shape, w, rows + 64, max_draft=8)
    prompt = si.uniform_tokens(seed, 0, rows, shape.vocab).numpy()
    ms = []
    for _ in range(iters + 2):
        sess.prefill(prompt)
        ms.append(sess.get_stats()["ms_prefill"])         # CUDA events around the pass, on its stream
    ms = sorted(ms[2:])
    d, hd = shape.d_model, shape.head_dim
    weights = layers * (2 * d * shape.n_heads * hd + 2 * d * shape.n_kv_heads * hd + 3 * d * shape.d_ff)
    flop = 4.0 * rows * weights                             # 2 per multiply-add, two bf16 terms per activation
    med = ms[len(ms) // 2]
    return {"op": "prompt", "shape": shape.name, "rows": rows, "ms_per_pass": med, "ms_min": ms[0],
            "linear_flop": flop, "tflops": flop / med / 1e9}


def bench_anchors(n_domains: int, per: int, d: int, iters: int, k: int = 10, seed: int = 3):
    build.build()
    from . import binding as kb
    torch.cuda.set_device(0)
    X = si.anchors(seed, n_domains, per, d, 0.5, normalise=False).cuda()
    init = X[:n_domains].contiguous()                        # all from the first domain: several rounds
    ms, rounds = [], 0
    for _ in range(iters + 2):
        r = kb.knnssd_build_anchors(X, init, 50, k)
        ms.append(r["ms_rounds"])
        rounds = r["rounds"]
    ms = sorted(ms[2:])
    med = ms[len(ms) // 2]
    nbytes = 2.0 * X.numel() * 4 * (rounds - 1) + X.numel() * 4       # the last round only assigns
    return {"op": "anchors", "points": X.shape[0], "d": d, "clusters": n_domains, "k": k, "rounds": rounds,
            "ms_rounds": med, "ms_per_round": med / rounds, "algorithmic_bytes": nbytes, "gbs": nbytes / med / 1e6,
            "points_bytes": X.numel() * 4}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["linear", "linear_tc", "pass", "prompt", "anchors"])
    ap.add_argument("--shape", default="llama13b")
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--context", type=int, default=1280)
    ap.add_argument("--n-out", type=int, default=131072)
    ap.add_argument("--n-in", type=int, default=5120)
    ap.add_argument("--rows", type=int, default=1)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp32"])
    a = ap.parse_args()
    if a.op == "linear_tc":
        print(json.dumps(bench_linear_tc(a.n_out, a.n_in, a.rows, a.iters, a.warmup)))
    elif a.op == "anchors":
        print(json.dumps(bench_anchors(a.n_out, a.rows, a.n_in, a.iters)))
    elif a.op == "prompt":
        print(json.dumps(bench_prompt(a.shape, a.layers, a.context, a.iters)))
    elif a.op == "pass":
        print(json.dumps(bench_pass(a.shape, a.layers, a.context, a.rows, a.iters)))
    else:
        print(json.dumps(bench_linear(a.n_out, a.n_in, a.rows, a.iters, a.warmup, a.dtype)))


if __name__ == "__main__":
    main()
