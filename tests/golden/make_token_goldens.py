#!/usr/bin/env python
"""Writes the expected token streams of the full-size workloads with the CPU oracle.

Test infrastructure: imports only ``oracle`` and ``synthetic_inputs`` (never the CUDA package); every stored value
is the oracle's own output on seeded synthetic inputs.  One JSON file per case under ``tests/golden/``; the
``-m gpu`` tests in ``tests/test_gpu_named_sizes.py`` rebuild the same inputs from the recipe stored in the file and
compare what ``knnssd_generate`` returns with it, token for token.

A case is one request on a full-depth, full-width model with the prompt length of its workload, plain random-init
weights (nothing damped), the workload's draft length, five per-domain skip masks and 5 x 10 anchors; the request's
pooled last hidden state picks the domain (Eq. (4)) and with it the mask.  The oracle needs seconds per pass on these
shapes, so ``max_new`` may be shorter than the workload's (the file says so in ``cut``); depth, width and prompt
length are never reduced.

    python tests/golden/make_token_goldens.py llama13b-k4:160 llama13b-k2:48 llama13b-k8:48
    python tests/golden/make_token_goldens.py --list
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import synthetic_inputs as si  # noqa: E402

N_DOMAINS, PER_DOMAIN, SIGMA_A = 5, 10, 0.2
N_SAMPLED = 64          # logit / pooled-vector entries stored per row

# name: shape, prompt length, workload's max_new, k, skipped attention / MLP sublayers, kind
CASES = {
    "llama7b-k4": dict(shape="llama7b", prompt=512, max_new=256, k=4, skip=(14, 15)),
    "llama13b-k4": dict(shape="llama13b", prompt=1024, max_new=512, k=4, skip=(19, 17)),
    "llama13b-k2": dict(shape="llama13b", prompt=1024, max_new=512, k=2, skip=(19, 17)),
    "llama13b-k8": dict(shape="llama13b", prompt=1024, max_new=512, k=8, skip=(19, 17)),
    "qwen14b-k4": dict(shape="qwen14b", prompt=2048, max_new=512, k=4, skip=(19, 19)),
    # acceptance-shaped extra (not one of the named workloads): output projections of the selected domain's skipped
    # sublayers scaled by gamma, so that accept counts span 0..k at full depth
    "llama13b-k4-shaped": dict(shape="llama13b", prompt=1024, max_new=512, k=4, skip=(19, 17), gamma=3e-4,
                               shaped_domain=2),
    # the mixed-domain stream on the 13B shape: the first request of each domain in stream order
    "stream13b": dict(shape="llama13b", stream=True, max_new=256, k=4, skip=(19, 17), pool=(23, 21), mix_ratio=1.0,
                      requests_per_domain=40, prompt_range=(128, 1024), per_domain_cases=1),
    # seconds-long cases on a small shape (three layers, widths that are multiples of 128): a check of this script
    "small-k4": dict(shape="stream-bf16", prompt=150, max_new=24, k=4, skip=(1, 1)),
    "small-stream": dict(shape="stream-bf16", stream=True, max_new=12, k=4, skip=(1, 1), pool=(2, 2), mix_ratio=1.0,
                         requests_per_domain=2, prompt_range=(20, 90), per_domain_cases=1),
}


def domain_masks(seed, shape, skip):
    return np.stack([si.skip_mask_split(seed + 100 + i, shape.n_layers, skip[0], skip[1]) for i in range(N_DOMAINS)])


def sampled_indices(seed, tag, n, size):
    return np.array(sorted({si.hash_u64_int(seed, si.TensorId.PROMPT - 1 - tag, j) % size for j in range(n)}), dtype=np.int64)


def cosines(v, anchors):
    v64, a64 = v.astype(np.float64), anchors.astype(np.float64)
    return (a64 @ v64) / (np.linalg.norm(a64, axis=1) * np.linalg.norm(v64))


def prefill_and_select(om, shape, prompt, query_of, anchors, seed, log):
    t0 = time.time()
    pooled, first, first_margin = om.prefill(prompt)
    log(f"prefill of {len(prompt)} rows: {time.time() - t0:.0f} s")
    query = query_of(pooled)
    dom, anc, cos = oracle.knn_select(query, anchors, N_DOMAINS, PER_DOMAIN)
    # how clear the choice of DOMAIN is (reported only; numpy here is bookkeeping, the choice itself is the oracle's)
    cs = cosines(query, anchors).reshape(N_DOMAINS, PER_DOMAIN).max(axis=1)
    pidx = sampled_indices(seed, 2, N_SAMPLED, shape.d_model)
    return {"prompt_len": len(prompt), "first_token": int(first), "first_margin": float(first_margin),
            "domain": int(dom), "anchor": int(anc), "cosine": float(cos),
            "domain_gap": float(np.sort(cs)[-1] - np.sort(cs)[-2]),
            "pooled_index": [int(i) for i in pidx], "pooled": [float(pooled[i]) for i in pidx],
            "pooled_norm": float(np.linalg.norm(pooled.astype(np.float64)))}


def generate_from_prompt_end(om, shape, head, mask, k, max_new, seed, log):
    """Decodes max_new tokens from the state the prompt pass left (the cache rows beyond the prompt are dead)."""
    P, first = head["prompt_len"], head["first_token"]
    om.length = P
    t0 = time.time()
    gen = om.generate(first, max_new, k, mask)
    log(f"k={k}: {max_new} tokens in {gen['rounds']} rounds, accepted {gen['accepted']}/{gen['drafted']}, "
        f"min margin {gen['min_margin']:.3e}: {time.time() - t0:.0f} s")
    # teacher-forced sample of the first verification pass: rows [first, drafts of round 0] at the prompt's end
    om.length = P
    rows = [first] + ([int(t) for t in gen["drafts"][0] if t >= 0] if gen["rounds"] and k > 0 else [])
    fw = om.forward(np.array(rows, dtype=np.int32), P, want_logits=True, want_hidden=False)
    idx = sampled_indices(seed, 1, N_SAMPLED, shape.vocab)
    out = dict(head)
    out.update({
        "tokens": [int(t) for t in gen["tokens"]], "accepts": [int(a) for a in gen["accepts"]],
        "rounds": int(gen["rounds"]), "drafted": int(gen["drafted"]), "accepted": int(gen["accepted"]),
        "min_margin": float(gen["min_margin"]),
        "verify_rows": rows, "logit_index": [int(i) for i in idx],
        "logits": [[float(fw["logits"][r, i]) for i in idx] for r in range(len(rows))],
        "verify_argmax": [int(a) for a in fw["argmax"]], "verify_margin": [float(m) for m in fw["margin"]]})
    return out


def one_request(om, shape, prompt, query_of, anchors, masks, k, max_new, seed, log):
    head = prefill_and_select(om, shape, prompt, query_of, anchors, seed, log)
    return generate_from_prompt_end(om, shape, head, masks[head["domain"]], k, max_new, seed, log)


def run_cases(specs, seed, out_dir):
    """specs: [(case name, max_new or 0)].  Several cases may be given when they share model, prompt and weights
    (the same shape with different draft lengths): the prompt pass is then run once."""
    c0 = CASES[specs[0][0]]
    key = lambda c: (c["shape"], c.get("prompt"), c.get("stream", False), c.get("gamma"), tuple(c["skip"]))  # noqa: E731
    assert all(key(CASES[n]) == key(c0) for n, _ in specs), "cases given together must share model, weights and prompt"
    assert not (c0.get("stream") and len(specs) > 1)
    shape = si.SHAPES[c0["shape"]]
    tag = "+".join(n for n, _ in specs)

    def log(msg):
        print(f"[{tag} seed {seed}] {msg}", flush=True)

    def record(name, max_new):
        c = CASES[name]
        return {"case": name, "shape": c["shape"], "seed": seed, "k": c["k"], "max_new": max_new,
                "workload_max_new": c["max_new"],
                "cut": None if max_new == c["max_new"] else
                f"generated length {max_new} instead of {c['max_new']} (oracle time); depth, width and prompt as named",
                "n_domains": N_DOMAINS, "anchors_per_domain": PER_DOMAIN, "sigma_a": SIGMA_A, "skip": list(c["skip"]),
                "written_by": "tests/golden/make_token_goldens.py (CPU oracle only)", "oracle_cores": os.cpu_count()}

    def write(rec, t0):
        rec["oracle_seconds"] = round(time.time() - t0)
        path = os.path.join(out_dir, f"tokens_{rec['case']}.json")
        with open(path, "w") as f:
            json.dump(rec, f)
            f.write("\n")
        log(f"wrote {path} after {rec['oracle_seconds']} s")

    lens = [min(m or CASES[n]["max_new"], CASES[n]["max_new"]) for n, m in specs]
    anchors = si.anchors(seed, N_DOMAINS, PER_DOMAIN, shape.d_model, SIGMA_A).numpy()
    t0 = time.time()
    if c0.get("stream"):
        name, max_new, c = specs[0][0], lens[0], c0
        rec = record(name, max_new)
        pool, masks = si.nested_skip_masks(seed + 100, shape.n_layers, N_DOMAINS, c["pool"][0], c["pool"][1],
                                           c["skip"][0], c["skip"][1])
        w = si.make_model_weights(shape, seed)
        log(f"weights: {time.time() - t0:.0f} s")
        per = c["requests_per_domain"]
        labels = si.request_stream(seed, N_DOMAINS, per, c["mix_ratio"])
        lengths = si.prompt_lengths(seed, N_DOMAINS * per, *c["prompt_range"])
        cen = si.domain_centroids(seed, N_DOMAINS, shape.d_model).numpy()
        seen, picked = {}, []
        for i, d in enumerate(labels):
            if seen.get(d, 0) < c["per_domain_cases"]:
                seen[d] = seen.get(d, 0) + 1
                picked.append(i)
        rec.update(mix_ratio=c["mix_ratio"], requests_per_domain=per, prompt_range=list(c["prompt_range"]),
                   pool=list(c["pool"]), requests=[],
                   subset=f"the first {c['per_domain_cases']} request(s) of each domain in stream order (oracle time)")
        om = oracle.OracleModel(shape, w, c["prompt_range"][1] + max_new + 16)
        for i in picked:
            prompt = si.uniform_tokens(seed, 1 + i, lengths[i], shape.vocab).numpy()
            cD = cen[labels[i]]

            def query_of(pooled, cD=cD):
                # a draw from the domain's cluster: the request's own pooled state shifted towards the centroid
                scale = 4.0 * np.linalg.norm(pooled.astype(np.float64)) / np.linalg.norm(cD.astype(np.float64))
                return (pooled + np.float32(scale) * cD).astype(np.float32)

            head = prefill_and_select(om, shape, prompt, query_of, anchors, seed, log)
            r = generate_from_prompt_end(om, shape, head, masks[head["domain"]], c["k"], max_new, seed, log)
            r.update(index=i, label=int(labels[i]))
            rec["requests"].append(r)
        write(rec, t0)
        return
    masks = domain_masks(seed, shape, c0["skip"])
    damp = None
    if "gamma" in c0:
        damp = {int(j): c0["gamma"] for j in np.nonzero(masks[c0["shaped_domain"]])[0]}
    w = si.make_model_weights(shape, seed, damp=damp)
    log(f"weights: {time.time() - t0:.0f} s")
    prompt = si.uniform_tokens(seed, 0, c0["prompt"], shape.vocab).numpy()
    om = oracle.OracleModel(shape, w, c0["prompt"] + max(lens) + 16)
    head = prefill_and_select(om, shape, prompt, lambda p: p, anchors, seed, log)
    for (name, _), max_new in zip(specs, lens):
        c = CASES[name]
        rec = record(name, max_new)
        dom = head["domain"]
        if "gamma" in c:
            # the request belongs to the shaped domain: the test sets that domain's mask explicitly
            dom = c["shaped_domain"]
            rec.update(gamma=c["gamma"], shaped_domain=dom, explicit_mask_domain=dom)
        rec["requests"] = [generate_from_prompt_end(om, shape, head, masks[dom], c["k"], max_new, seed, log)]
        write(rec, t0)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("cases", nargs="*", help="case[:max_new] ...; cases given together share one prompt pass")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--list", action="store_true")
    ap.add_argument("--out-dir", default=HERE)
    a = ap.parse_args()
    if a.list or not a.cases:
        for n, c in CASES.items():
            print(n, c)
        return
    specs = [(s.split(":")[0], int(s.split(":")[1]) if ":" in s else 0) for s in a.cases]
    run_cases(specs, a.seed, a.out_dir)


if __name__ == "__main__":
    main()
