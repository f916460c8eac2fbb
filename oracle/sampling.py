"""Stochastic speculative sampling - CPU oracle (test infrastructure only).

Only ``tests/``, the smoke check and the benchmark's CPU-baseline leg may import this module; it imports nothing from
the CUDA package.  Plain numpy in fp64, pure-Python loops.

What the paper fixes: the decoding set-up lists temperature 0.2 and top-p 0.85 (App. C.1) beside the greedy setting of
Table 1, and the method is said to leave the distribution of the generated tokens unchanged (Sec. 1, Sec. 3.1).  It
prints no acceptance rule for the sampled case.  Reading taken here: the rule of speculative sampling that has exactly
that property -

* p and q are the full model's and the draft model's next-token distributions AFTER temperature and top-p filtering
  (``filtered_distribution``);
* a drafted token d ~ q is kept with probability min(1, p(d) / q(d));
* at the first rejection the token is drawn instead from the normalised positive part of p - q, and the round ends;
* if all k drafts are kept, one more token is drawn from the full model's distribution after the last draft.

Random numbers are inputs: every draw consumes one uniform u in [0, 1) handed in by the caller, through the inverse
CDF taken in token-id order (``sample``), so that another implementation fed the same uniforms makes the same choices.

Pinned in ``tests/test_oracle_sampling.py``: temperature / top-p filtering against the transformer library's logits
warpers and hand-made closed forms; temperature -> 0 gives the greedy token; the emitted distribution equals p by
integration over the uniforms on small vocabularies; ``sample`` against ``numpy.searchsorted`` on the CDF.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def filtered_distribution(logits: Sequence[float], temperature: float, top_p: float) -> np.ndarray:
    """softmax(logits / temperature), then nucleus filtering: tokens are ranked by probability (highest first, lower
    id first among equals) and a token is kept iff the total probability of the tokens ranked before it is below
    ``top_p`` (so the kept set is the shortest prefix of that ranking whose mass reaches top_p, and never empty); the
    kept probabilities are renormalised to sum to one.  fp64 [V]."""
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    z = z - z.max()
    p = np.exp(z)
    p = p / p.sum()
    order = sorted(range(len(p)), key=lambda i: (-p[i], i))
    keep = np.zeros(len(p), dtype=bool)
    before = 0.0
    for i in order:
        if before < top_p:
            keep[i] = True
        before += p[i]
    out = np.where(keep, p, 0.0)
    return out / out.sum()


def nucleus_margin(logits: Sequence[float], temperature: float, top_p: float) -> float:
    """How far the kept / dropped decision of the nucleus filter is from flipping: the smallest |mass ranked before a
    token - top_p| over all tokens (reported so that tests can tell a rounding-sensitive row from a wrong one)."""
    z = np.asarray(logits, dtype=np.float64) / float(temperature)
    z = z - z.max()
    p = np.exp(z)
    p = p / p.sum()
    order = sorted(range(len(p)), key=lambda i: (-p[i], i))
    before, best = 0.0, np.inf
    for i in order:
        best = min(best, abs(before - top_p))
        before += p[i]
    return float(best)


def sample(weights: Sequence[float], u: float) -> int:
    """Inverse CDF in token-id order on non-negative weights (not necessarily normalised): the smallest id x with
    w_0 + .. + w_x > u * sum(w).  With u in [0, 1) and a positive total this always exists."""
    w = np.asarray(weights, dtype=np.float64)
    target = float(u) * float(w.sum())
    acc = 0.0
    last = -1
    for x in range(len(w)):
        if w[x] > 0.0:
            last = x
        acc += w[x]
        if acc > target:
            return x
    return last          # u * total rounded up to the total itself: the last token with weight


def sample_gap(weights: Sequence[float], u: float) -> float:
    """Distance (in units of the total weight) between the draw u and the nearest step of the CDF."""
    w = np.asarray(weights, dtype=np.float64)
    cdf = np.cumsum(w) / w.sum()
    return float(np.abs(cdf - u).min())


def accept_or_resample(p: Sequence[Sequence[float]], q: Sequence[Sequence[float]], drafts: Sequence[int],
                       u_accept: Sequence[float], u_final: float) -> Tuple[int, int]:
    """One verification round.  p [k+1][V]: the full model's filtered distributions after [pending], [pending, d_0], ..;
    q [k][V]: the draft model's filtered distributions the drafts were drawn from; drafts [k]; u_accept [k] and u_final
    uniforms.  Returns (n_accepted, next_token): draft j is kept iff u_accept[j] * q_j(d_j) < p_j(d_j); at the first
    rejected j the next token is ``sample(max(0, p_j - q_j), u_final)``; with all k kept it is ``sample(p_k, u_final)``."""
    k = len(drafts)
    for j in range(k):
        pj, qj = np.asarray(p[j], dtype=np.float64), np.asarray(q[j], dtype=np.float64)
        d = int(drafts[j])
        if float(u_accept[j]) * qj[d] < pj[d]:
            continue
        resid = np.maximum(pj - qj, 0.0)
        if not resid.sum() > 0.0:      # p == q exactly: nothing to resample from; the draft's own distribution stands
            resid = pj
        return j, sample(resid, u_final)
    return k, sample(np.asarray(p[k], dtype=np.float64), u_final)


def accept_margin(p, q, drafts, u_accept) -> float:
    """Smallest |u q(d) - p(d)| over the drafts that were examined (how close a keep / reject decision was)."""
    best = np.inf
    for j, d in enumerate(drafts):
        a, b = float(u_accept[j]) * float(q[j][int(d)]), float(p[j][int(d)])
        best = min(best, abs(a - b))
        if not a < b:
            break
    return float(best)


def generate_sampled(model, first_token: int, max_new: int, k: int, skip_mask, temperature: float, top_p: float,
                     uniforms: Sequence[float]):
    """The draft-and-verify loop (Sec. 4.2) with sampled decoding on an ``oracle.OracleModel`` that has been prefilled.
    Emits exactly max_new tokens, the first being ``first_token``.  Round r uses uniforms[r (2k + 1) + j] for the draw
    of draft j, [r (2k + 1) + k + j] for its keep test and [r (2k + 1) + 2k] for the round's last draw.  Returns
    dict(tokens, accepts, margin): margin = how close any decision of the run came to flipping (the smallest of the
    nucleus margins, the draw gaps and the keep-test margins), for tests that compare another implementation."""
    stride = 2 * k + 1
    tokens: List[int] = [int(first_token)]
    accepts: List[int] = []
    pending, n, rnd, margin = int(first_token), model.length, 0, np.inf
    while len(tokens) < max_new:
        keff = min(k, max_new - len(tokens) - 1)
        u = uniforms[rnd * stride:(rnd + 1) * stride]
        q, drafts, cur = [], [], pending
        for j in range(keff):
            lg = model.forward([cur], n + j, skip_mask=skip_mask)["logits"][0]
            qj = filtered_distribution(lg, temperature, top_p)
            d = sample(qj, u[j])
            margin = min(margin, nucleus_margin(lg, temperature, top_p), sample_gap(qj, u[j]))
            q.append(qj)
            drafts.append(d)
            cur = d
        lgs = model.forward([pending] + drafts, n)["logits"]
        p = [filtered_distribution(lgs[j], temperature, top_p) for j in range(keff + 1)]
        a, nxt = accept_or_resample(p, q, drafts, u[k:k + keff], u[2 * k])
        for j in range(keff + 1):
            margin = min(margin, nucleus_margin(lgs[j], temperature, top_p))
        if keff:
            margin = min(margin, accept_margin(p, q, drafts, u[k:k + keff]))
        resid = np.maximum(p[a] - q[a], 0.0) if a < keff else p[keff]
        margin = min(margin, sample_gap(resid if resid.sum() > 0 else p[a], u[2 * k]))
        tokens.extend(drafts[:a] + [nxt])
        accepts.append(a)
        pending = nxt
        n += a + 1
        model.length = n
        rnd += 1
    return {"tokens": np.array(tokens, dtype=np.int32), "accepts": np.array(accepts, dtype=np.int32), "margin": float(margin)}
