#!/usr/bin/env python
"""Benchmark of the KNN-SSD decode hot path on B200 (one replica per GPU; requests are independent).

Workload (default): LLaMA-2-13B-shaped decoder, bf16 random-init weights, a 1024-token random prompt, 512 new tokens,
draft length k = 4, a seeded skip mask dropping 19 attention + 17 MLP sublayers of 80 (45 %), 5 domains x 10 anchors.
A "step" is one request's decode hot path with the prompt already resident (KV cache filled): cosine selection of the
skip mask, then rounds of k draft passes + one verification pass + accept/rollback until 512 tokens are out.
``value`` = emitted tokens / s over the timed steps (device-resident inputs); ``e2e`` = the same through
knnssd_generate with the prompt in host memory (prefill, copies and read-backs inside the timed region).  Both are
measured on the workload as written: plain random-init weights, on which almost no draft is accepted, so they are the
rate of one token per round.  What does not depend on acceptance - the latency and the HBM rate of the draft pass and
of the verification passes for k = 2, 4, 8 - is in ``passes`` and ``roofline``; ``tokens_per_s_by_accepted_drafts``
gives the rate those latencies imply for every accept length, and ``acceptance_shaped`` is a labelled synthetic
scenario (skipped sublayers damped) in which drafts are accepted about as often as in the paper's tables.

`--impl reference` times the CPU oracle (the stand-in for a reference implementation in this build) on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synthetic_inputs as si  # noqa: E402

METRIC = "decode tokens/s at batch 1 (self-speculative: k draft passes + 1 verify pass per round)"
UNIT = "tokens/s"

WORKLOADS = {
    # name: (shape, prompt_len, max_new, n_attn_skip, n_mlp_skip)
    "llama13b": ("llama13b", 1024, 512, 19, 17),
    "llama7b": ("llama7b", 512, 256, 14, 15),
    "qwen14b": ("qwen14b", 2048, 512, 19, 19),
    "tiny": ("tiny", 32, 32, 1, 2),
}
N_DOMAINS, PER_DOMAIN = 5, 10
REQUEST_DOMAIN = 2          # the synthetic request is drawn from this domain's cluster


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def prompt_pass_report(shape, rows, ms_list):
    ms = sorted(ms_list)[len(ms_list) // 2]
    d, hd = shape.d_model, shape.head_dim
    weights = shape.n_layers * (2 * d * shape.n_heads * hd + 2 * d * shape.n_kv_heads * hd + 3 * d * shape.d_ff)
    flop = 4.0 * rows * weights          # executed: every activation is two bf16 terms
    out = {"rows": rows, "ms": ms, "linear_tflops_executed": flop / ms / 1e9,
           "linear_tflops_algorithmic": 0.5 * flop / ms / 1e9, "bound": "tensor"}
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            pk = json.load(f)
        out["peak_bf16_tflops_sustained"] = pk.get("bf16_tflops_sustained")
        if pk.get("bf16_tflops_sustained"):
            out["frac_of_measured_sustained"] = out["linear_tflops_executed"] / pk["bf16_tflops_sustained"]
            out["frac_algorithmic"] = out["linear_tflops_algorithmic"] / pk["bf16_tflops_sustained"]
    return out


def pass_bytes(shape, mask, n_ctx, rows):
    """Algorithmic bytes of one pass: weights of the retained sublayers + LM head + K/V rows attended."""
    b = 2 if shape.dtype == "bf16" else 4
    d, hd = shape.d_model, shape.head_dim
    attn_w = (2 * d * shape.n_heads * hd + 2 * d * shape.n_kv_heads * hd) * b
    mlp_w = 3 * d * shape.d_ff * b
    head_w = shape.vocab * d * b
    kv = 2 * shape.n_kv_heads * hd * b * (n_ctx + rows)
    n_attn = sum(1 for l in range(shape.n_layers) if mask is None or not mask[2 * l])
    n_mlp = sum(1 for l in range(shape.n_layers) if mask is None or not mask[2 * l + 1])
    weights = n_attn * attn_w + n_mlp * mlp_w + head_w
    return weights, n_attn * kv


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "200", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for nme, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nme)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def build_inputs(workload: str, seed: int, device, gamma: float):
    shape_name, prompt_len, max_new, na, nm = WORKLOADS[workload]
    shape = si.SHAPES[shape_name]
    masks = np.stack([si.skip_mask_split(seed + 100 + i, shape.n_layers, na, nm) for i in range(N_DOMAINS)])
    anchors = si.anchors(seed, N_DOMAINS, PER_DOMAIN, shape.d_model, 0.2)
    prompt = si.uniform_tokens(seed, 0, prompt_len, shape.vocab).numpy()
    return shape, masks, anchors, prompt, max_new


def reduce_over_replicas(ms, e2e_s, tokens, e2e_tokens, launches, device, world):
    """Whole-job figures of N independent replicas (one per GPU, no traffic between them while they work): the slowest
    replica sets the time (MAX over ranks), work adds up (SUM over ranks)."""
    if world <= 1:
        return ms, e2e_s, tokens, e2e_tokens, launches
    import torch.distributed as dist
    t = torch.tensor([ms, e2e_s], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([tokens, e2e_tokens, launches], device=device, dtype=torch.float64)
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), int(c[0]), int(c[1]), int(c[2])


def damp_in_place(shape, w, seed, sublayers, gamma, dev):
    """Regenerates the output projections (W_o / W_down) of the given sublayers with their standard deviation scaled
    by gamma: the "acceptance-shaped" weights (same shapes, same bytes)."""
    d, hq, f, s = shape.d_model, shape.n_heads * shape.head_dim, shape.d_ff, shape.sigma
    for j in sublayers:
        l, t = j // 2, si.TensorId.LAYER0 + 8 * (j // 2)
        if j % 2 == 0:
            w["wo"][l] = si.normal_weight(seed, t + 3, d, hq, s * gamma, shape.dtype, dev)
        else:
            w["w_down"][l] = si.normal_weight(seed, t + 6, d, f, s * gamma, shape.dtype, dev)


def run_scenario(kb, args, shape, w, masks, anchors, prompt, max_new, k, dev, world, rank, local, steps, warmup, e2e_steps,
                 extra_ks=()):
    """One request shape measured two ways: the decode hot path with the prompt's K/V resident (CUDA events), and the
    whole request through knnssd_generate with host buffers (wall clock around synchronised calls)."""
    max_seq = len(prompt) + max_new + 64
    # Domains are Gaussian clusters in hidden space and a request is a draw from its domain's cluster.  The request's
    # pooled last-layer state is whatever this random-init model produces for the prompt, so the cluster of
    # REQUEST_DOMAIN is centred there: a first session (no anchors) yields that state, then the anchors are drawn.
    probe = kb.Session.from_shape(shape, w, max_seq, max_draft=max(k, 8))
    _, pooled0 = probe.prefill(prompt, want_pooled=True)
    probe.close()
    anchors = anchors.to(dev).clone()
    unit = pooled0 / pooled0.norm()
    lo, hi = REQUEST_DOMAIN * PER_DOMAIN, (REQUEST_DOMAIN + 1) * PER_DOMAIN
    noise = si.normal_f32(args.seed, si.TensorId.ANCHOR + 1000, torch.arange(PER_DOMAIN * shape.d_model, device=dev), 1.0)
    own = unit[None, :] + 0.2 / (shape.d_model ** 0.5) * noise.view(PER_DOMAIN, shape.d_model)
    anchors[lo:hi] = own / own.norm(dim=1, keepdim=True)
    sess = kb.Session.from_shape(shape, w, max_seq, max_draft=max(k, 8), anchors=anchors.contiguous(), skip_masks=masks,
                                 anchors_per_domain=PER_DOMAIN)
    first, pooled = sess.prefill(prompt, want_pooled=True)
    query = pooled
    dom, anc, cos = sess.select_skipset(query)
    if dom != REQUEST_DOMAIN:
        raise SystemExit(f"selection picked domain {dom}, expected {REQUEST_DOMAIN}")
    P = len(prompt)

    def decode_step():
        sess.set_length(P)
        sess.set_pending(first)
        sess.select_skipset(query)
        return sess.decode(max_new, k)

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()

    for _ in range(warmup):
        r = decode_step()
    sync_all()
    sampler = ClockSampler(local) if rank == 0 else None
    l0 = sess.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    tokens = 0
    for _ in range(steps):
        r = decode_step()
        tokens += len(r["tokens"])
    e1.record()
    sync_all()
    out = {"ms": e0.elapsed_time(e1), "tokens": tokens, "launches": sess.launch_count - l0, "stats": r["stats"],
           "accepts": r["accepts"], "dom": dom, "sess": sess, "P": P}
    # per-pass latency at mid-generation context
    sess.set_length(min(sess.length, P + max_new // 2))
    out["n_mid"] = sess.length
    out["t_draft"] = sess.time_pass(0, k, args.pass_iters)
    out["t_verify"] = sess.time_pass(1, k, args.pass_iters)
    out["t_verify_extra"] = {kk: sess.time_pass(1, kk, args.pass_iters) for kk in extra_ks if kk != k}
    out["clocks"] = sampler.stop() if sampler else None
    # end to end through the public call with host buffers
    sess.generate(prompt, max_new, k, use_selection=True)
    sync_all()
    te = time.perf_counter()
    e2e_tokens, rounds_e2e, prefill_ms = 0, 0, []
    for _ in range(e2e_steps):
        rr = sess.generate(prompt, max_new, k, use_selection=True)
        e2e_tokens += len(rr["tokens"])
        rounds_e2e += rr["stats"]["rounds"]
        prefill_ms.append(rr["stats"]["ms_prefill"])
    torch.cuda.synchronize()
    out.update(e2e_s=time.perf_counter() - te, e2e_tokens=e2e_tokens, rounds_e2e=rounds_e2e, prefill_ms=prefill_ms,
               e2e_steps=e2e_steps)
    return out


def pass_record(nbytes, t, peak, rows):
    ms = t["ms_per_pass"]
    gbs = nbytes / ms / 1e6
    return {"rows": rows, "ms": ms, "gbs": gbs, "frac_of_peak": gbs / peak, "frac_of_8TBs": gbs / 8000.0, "launches": t["launches"]}


def run_ours(args):
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding as kb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    shape, masks, anchors, prompt, max_new = build_inputs(args.workload, args.seed, dev, args.gamma)
    k = args.k
    t0 = time.time()
    # the workload as written: plain random-init weights (gamma = 1).  gamma < 1 damps the output projections of the
    # sublayers that the request's domain mask skips (see the acceptance-shaped scenario below)
    damp = None
    if args.gamma < 1.0:
        damp = {int(j): args.gamma for j in np.nonzero(masks[REQUEST_DOMAIN])[0]}
    w = si.make_model_weights(shape, args.seed, device=dev, damp=damp)
    torch.cuda.synchronize()
    t_weights = time.time() - t0
    e2e_steps = max(1, min(args.steps, 2))
    sc = run_scenario(kb, args, shape, w, masks, anchors, prompt, max_new, k, dev, world, rank, local, args.steps, args.warmup,
                      e2e_steps, extra_ks=(2, 4, 8) if shape.dtype == "bf16" else ())
    sess, dom, P, n_mid = sc["sess"], sc["dom"], sc["P"], sc["n_mid"]
    mask = masks[dom]
    stats, accepts, t_draft, t_verify, clocks = sc["stats"], sc["accepts"], sc["t_draft"], sc["t_verify"], sc["clocks"]
    ms, e2e_s, tokens, e2e_tokens, launches = reduce_over_replicas(sc["ms"], sc["e2e_s"], sc["tokens"], sc["e2e_tokens"],
                                                                   sc["launches"], dev, world)
    rounds_e2e, prefill_ms = sc["rounds_e2e"], sc["prefill_ms"]
    if rank != 0:
        return
    peak, peak_kind = peaks()
    wd, kvd = pass_bytes(shape, mask, n_mid, 1)
    wv, kvv = pass_bytes(shape, None, n_mid, k + 1)
    # dominant kernel: the persistent pass kernel (one launch per draft step, one per verification pass).
    # algorithmic bytes of a launch = weights of the sublayers it runs + LM head + K/V rows it attends.
    round_bytes = k * (wd + kvd) + (wv + kvv)
    round_ms = k * t_draft["ms_per_pass"] + t_verify["ms_per_pass"]
    achieved = round_bytes / (round_ms * 1e-3) / 1e9
    # DRAM traffic per launch: counters were taken on a 4-layer capture of the same kernel (profiles/); every weight
    # byte is read once per pass, so the measured traffic / algorithmic ratio carries over to the full list
    traffic = None
    tp = os.path.join(ROOT, "profiles", "pass_kernel_traffic.json")
    if os.path.exists(tp) and shape.dtype == "bf16":
        with open(tp) as f:
            tr = json.load(f)
        traffic = (k * (wd + kvd) * tr["ratio_rows1"] + (wv + kvv) * tr["ratio_rows5"]) / (k + 1)
    from paper_2505_16162_b200 import metrics
    n_skip = int(mask.sum())
    M_len = metrics.mean_generated_length(accepts) if len(accepts) else 1.0
    alpha = stats["accepted"] / stats["drafted"] if stats["drafted"] else 0.0
    passes = {"context": n_mid, "draft": pass_record(wd + kvd, t_draft, peak, 1),
              "verify": {f"k{k}": pass_record(wv + kvv, t_verify, peak, k + 1)},
              # kept under their old names for readers of earlier records
              "draft_ms": t_draft["ms_per_pass"], "verify_ms": t_verify["ms_per_pass"],
              "draft_frac_of_peak": (wd + kvd) / t_draft["ms_per_pass"] / 1e6 / peak,
              "verify_frac_of_peak": (wv + kvv) / t_verify["ms_per_pass"] / 1e6 / peak}
    for kk, tv in sc["t_verify_extra"].items():
        wk, kvk = pass_bytes(shape, None, n_mid, kk + 1)
        passes["verify"][f"k{kk}"] = pass_record(wk + kvk, tv, peak, kk + 1)
    # tokens/s the two pass times give for a accepted drafts per round, a = 0 .. k (Sec. 4.2: a + 1 tokens per round)
    closed_form = {f"a{a}": (a + 1) / (round_ms * 1e-3) for a in range(k + 1)}
    out = {
        "metric": METRIC, "value": tokens / (ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32 accumulate over bf16 weights" if shape.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": f"{args.workload}: {shape.n_layers} layers d={shape.d_model} ff={shape.d_ff} "
                               f"V={shape.vocab}, prompt {P}, {max_new} new tokens, k={k}, mask skips "
                               f"{n_skip}/{2 * shape.n_layers} sublayers, {N_DOMAINS}x{PER_DOMAIN} anchors",
                   "weights": "random init N(0,0.02) " + shape.dtype + (f"; output projections of mask-skipped sublayers scaled by {args.gamma} (acceptance-shaped)" if args.gamma < 1 else " (as the workload is written: nothing damped)"),
                   "l2": "inputs (weights) far larger than L2, no flush needed", "replicas": world,
                   "selected_domain": dom},
        "gpu_launches": launches,
        "e2e": {"value": e2e_tokens / e2e_s, "unit": UNIT,
                "h2d_bytes_per_step": int(P * 4), "d2h_bytes_per_step": int(max_new * 4 + (rounds_e2e // e2e_steps) * 20 + 16)},
        "roofline": {"bound": "hbm", "kernel": "pass_kernel (one decoder pass: weight-streaming linears + KV attention + head)",
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "bytes_per_launch": round_bytes / (k + 1),
                     "launch_mix": f"{k} draft passes (1 row) + 1 verify pass ({k + 1} rows) per round, CUDA events per pass"},
        "passes": passes,
        "tokens_per_s_by_accepted_drafts": closed_form,
        "acceptance": {"mean_generated_length": M_len, "alpha": alpha, "rounds": stats["rounds"],
                       "expected_speedup_c_plain": metrics.expected_speedup(M_len, alpha, metrics.cost_coefficient(n_skip / (2 * shape.n_layers))) if alpha > 0 else None},
        # the prompt pass inside the end-to-end steps (CUDA events around it): every linear map is one tensor-core
        # contraction over all prompt rows, activations as two bf16 terms, so 4 x rows x weights FLOP are executed
        # for the 2 x rows x weights the method asks for
        "prompt_pass": prompt_pass_report(shape, P, prefill_ms),
        "setup_s": {"weights": t_weights},
        "clocks": clocks,
    }
    if world == 1:
        out["anchor_construction"] = anchor_construction_report(shape, args.seed, dev, peak, not args.no_cpu_baseline)
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(args, shape, w, masks[dom], steps=1, warmup=0, sess=sess)
    if world == 1 and args.gamma >= 1.0 and args.shaped_gamma > 0 and shape.dtype == "bf16":
        # A synthetic scenario beside the workload as written, NOT comparable with the paper's tables: a random-init
        # model accepts almost no draft once 45 % of its sublayers are dropped, while the method presumes that a domain's
        # skippable sublayers matter little for it.  Here the output projections of the sublayers in the request's
        # domain mask are scaled by shaped_gamma (same shapes, same bytes, same pass latencies), so that the loop runs
        # at accept lengths like the paper's (alpha 0.85-1.0).
        sess.close()
        damp_in_place(shape, w, args.seed, [int(j) for j in np.nonzero(masks[REQUEST_DOMAIN])[0]], args.shaped_gamma, dev)
        s2 = run_scenario(kb, args, shape, w, masks, anchors, prompt, max_new, k, dev, 1, 0, local, args.steps, 1, 1)
        st2 = s2["stats"]
        out["acceptance_shaped"] = {
            "note": "synthetic scenario: output projections of the mask-skipped sublayers scaled by gamma; same bytes and pass latencies",
            "gamma": args.shaped_gamma, "alpha": st2["accepted"] / max(1, st2["drafted"]),
            "mean_generated_length": metrics.mean_generated_length(s2["accepts"]) if len(s2["accepts"]) else 1.0,
            "tokens_per_s": s2["tokens"] / (s2["ms"] * 1e-3), "e2e_tokens_per_s": s2["e2e_tokens"] / s2["e2e_s"],
            "draft_ms": s2["t_draft"]["ms_per_pass"], "verify_ms": s2["t_verify"]["ms_per_pass"]}
        s2["sess"].close()
    print(json.dumps(out))


def anchor_construction_report(shape, seed, dev, hbm_peak, with_oracle):
    """The pre-inference step that makes the anchors (not part of the timed decode step): K-means over N_DOMAINS x 1000
    synthetic pooled vectors of the model's width from a start inside one domain, 10 anchors per cluster; device time
    of the rounds' kernels, and the oracle's wall time on the same input with the results compared."""
    from paper_2505_16162_b200 import binding as kb
    per, k_anchor = 1000, 10
    X = si.anchors(seed + 3, N_DOMAINS, per, shape.d_model, 0.5, normalise=False).to(dev)
    init = X[:N_DOMAINS].contiguous()
    res = [kb.knnssd_build_anchors(X, init, 50, k_anchor) for _ in range(5)]
    ms = sorted(r["ms_rounds"] for r in res[2:])[1]
    rounds = res[-1]["rounds"]
    nbytes = X.numel() * 4 * (2 * (rounds - 1) + 1)          # a round reads the points twice; the last only assigns
    out = {"points": int(X.shape[0]), "d": shape.d_model, "clusters": N_DOMAINS, "anchors_per_cluster": k_anchor, "rounds": rounds,
           "ms_rounds": ms, "gbs": nbytes / ms / 1e6, "frac_of_hbm_peak": nbytes / ms / 1e6 / hbm_peak,
           "note": "the points (102 MB at d = 5120) mostly stay in L2 between the two reads of a round"}
    if with_oracle:
        from oracle import anchors as oa
        t0 = time.perf_counter()
        want = oa.build_anchors(X.cpu().numpy(), init.cpu().numpy().astype(np.float64), 50, k_anchor)
        out["oracle_s"] = time.perf_counter() - t0
        out["gpu_matches_oracle"] = bool(np.array_equal(want["labels"], res[-1]["labels"]) and
                                         np.array_equal(want["anchors"], res[-1]["anchors"]) and want["rounds"] == rounds)
    return out


def cpu_baseline(args, shape, w_dev, mask, steps, warmup, per_step=None, sess=None):
    """The oracle as it stands, on this host's cores, on a bounded sample: a short prompt and a few rounds.  With a
    session given, the CUDA path runs the same sample at full model size and the two token streams are compared."""
    import oracle
    w = {kname: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for kname, v in w_dev.items()}
    sp, sn = args.cpu_prompt, args.cpu_new
    prompt = si.uniform_tokens(args.seed, 0, sp, shape.vocab).numpy()
    om = oracle.OracleModel(shape, w, sp + sn * (warmup + steps) + args.k + 8)
    _, first, _ = om.prefill(prompt)
    times = []
    for i in range(warmup + steps):
        t0 = time.perf_counter()
        r = om.generate(first, sn, args.k, mask)
        dt = time.perf_counter() - t0
        first = int(r["tokens"][-1])
        if i >= warmup:
            times.append(dt)
        if per_step:
            per_step(dt)
    total = sum(times)
    out = {"value": sn * len(times) / total, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
           "sample": f"same shape and mask, {sp}-token prompt, {sn} new tokens per step with k={args.k} "
                     f"({len(times)} timed step(s), decode only)", "ms_per_step": 1e3 * total / len(times)}
    if sess is not None and warmup == 0 and steps == 1:
        # full-size parity on the sample: same prompt, mask and k through the CUDA path
        sess.set_skipmask(mask)
        g = sess.generate(prompt, sn, args.k)
        out["gpu_matches_oracle_on_sample"] = bool(np.array_equal(g["tokens"], r["tokens"]) and
                                                   np.array_equal(g["accepts"], r["accepts"]))
    return out


def run_stream(args):
    """Mixed-domain request stream on the 13B shape (the fifth workload): requests drawn from 5 synthetic domains, the
    order given by the mix-ratio chain (Sec. 4.2), prompts of 128-1024 random tokens; per request: prefill, the
    request's pooled state shifted into its domain's cluster, cosine selection of the skip mask, 256 tokens of
    self-speculative decoding with k = 4.  The domains' masks are drawn from one pool of sublayers whose output
    projections are scaled by gamma (what the method presumes of skippable sublayers)."""
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding as kb
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    shape = si.SHAPES["llama13b"]
    per = args.stream_requests // N_DOMAINS
    n_req, k, max_new = per * N_DOMAINS, 4, 256
    pool, masks = si.nested_skip_masks(args.seed + 100, shape.n_layers, N_DOMAINS, 23, 21, 19, 17)
    damp = {int(j): args.gamma for j in np.nonzero(pool)[0]} if args.gamma < 1.0 else None
    w = si.make_model_weights(shape, args.seed, device=dev, damp=damp)
    anchors = si.anchors(args.seed, N_DOMAINS, PER_DOMAIN, shape.d_model, 0.2).to(dev)
    cen = si.domain_centroids(args.seed, N_DOMAINS, shape.d_model).to(dev)
    labels = si.request_stream(args.seed, N_DOMAINS, per, args.mix_ratio)
    lengths = si.prompt_lengths(args.seed, n_req, 128, 1024)
    sess = kb.Session.from_shape(shape, w, 1024 + max_new + 64, max_draft=8, anchors=anchors, skip_masks=masks,
                                 anchors_per_domain=PER_DOMAIN)
    sel_ms, pre_ms, draft_ms, verify_ms, alphas, mlen, correct, tokens = [], [], [], [], [], [], 0, 0
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(n_req):
        prompt = si.uniform_tokens(args.seed, 1 + i, lengths[i], shape.vocab).numpy()
        _, pooled = sess.prefill(prompt, want_pooled=True)
        c = cen[labels[i]]
        query = (pooled + 4.0 * pooled.norm() / c.norm() * c).contiguous()     # a draw from the domain's cluster
        dom, _, _ = sess.select_skipset(query)
        r = sess.decode(max_new, k)
        st = r["stats"]
        correct += int(dom == labels[i])
        tokens += len(r["tokens"])
        sel_ms.append(st["ms_select"]); pre_ms.append(st["ms_prefill"])
        draft_ms.append(st["ms_draft"] / max(1, st["drafted"])); verify_ms.append(st["ms_verify"] / max(1, st["rounds"]))
        alphas.append(st["accepted"] / max(1, st["drafted"])); mlen.append(len(r["tokens"]) / max(1, st["rounds"]))
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    med = statistics.median
    print(json.dumps({
        "workload": f"stream13b: {n_req} requests from {N_DOMAINS} domains, mix ratio {args.mix_ratio}, prompts 128-1024, "
                    f"{max_new} new tokens, k={k}, gamma={args.gamma}",
        "domain_accuracy": correct / n_req, "tokens_per_s_incl_prefill": tokens / wall, "wall_s": wall,
        "select_ms_median": med(sel_ms), "select_ms_max": max(sel_ms), "prefill_ms_median": med(pre_ms),
        "draft_pass_ms_median": med(draft_ms), "verify_pass_ms_median": med(verify_ms),
        "alpha_mean": sum(alphas) / n_req, "alpha_min": min(alphas), "mean_generated_length": sum(mlen) / n_req,
        "switches": sum(1 for a, b in zip(labels, labels[1:]) if a != b)}))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape, masks, anchors, prompt, max_new = build_inputs(args.workload, args.seed, "cpu", 1.0)
    dev = torch.device("cuda", 0) if torch.cuda.is_available() else torch.device("cpu")
    damp = None
    if args.gamma < 1.0:
        damp = {int(j): args.gamma for j in np.nonzero(masks[REQUEST_DOMAIN])[0]}
    w = si.make_model_weights(shape, args.seed, device=dev, damp=damp)   # integer-only generator: same bits on any device
    cb = cpu_baseline(args, shape, w, masks[REQUEST_DOMAIN], steps=args.steps, warmup=args.warmup)
    out = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": cb["ms_per_step"], "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64 accumulate, f32 values", "data": "synthetic",
           "config": {"workload": f"{args.workload}: bounded sample of the same workload ({cb['sample']})"},
           "cpu_baseline": cb,
           "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama13b", choices=sorted(WORKLOADS))
    ap.add_argument("--k", type=int, default=4)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--gamma", type=float, default=1.0,
                    help="scale of the output projections of mask-skipped sublayers for the headline run (1 = plain random "
                         "init, the workload as written)")
    ap.add_argument("--shaped-gamma", type=float, default=0.0003,
                    help="the same scale for the labelled acceptance-shaped scenario reported beside the headline (0 = skip it)")
    ap.add_argument("--pass-iters", type=int, default=50)
    ap.add_argument("--cpu-prompt", type=int, default=16)
    ap.add_argument("--cpu-new", type=int, default=6)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stream-requests", type=int, default=0,
                    help="run the mixed-domain request stream (fifth workload) with this many requests instead of the bench")
    ap.add_argument("--mix-ratio", type=float, default=1.0)
    args = ap.parse_args()
    if args.stream_requests > 0:
        run_stream(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
