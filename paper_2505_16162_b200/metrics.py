"""Reporting utilities of the evaluation protocol (host side, no GPU work).

Mean generated length M, acceptance rate alpha and the expected wall-time
speed-up E(Spd.) = M*alpha / ((M - 1)*c + alpha)  [Sec. 5.1 "Evaluation
Metrics"; App. C.2, Eq. (7)], with the cost coefficient c either 1 - s (s = share
of skipped sublayers) or the refined form that weighs attention and MLP
sublayers by their latency ratio beta  [App. C.2, Eq. (8)].
"""
from __future__ import annotations

from typing import Sequence


def mean_generated_length(accepts: Sequence[int]) -> float:
    """M: tokens produced per full-model pass = mean over rounds of (accepted + 1)  [App. C.2]."""
    return sum(a + 1 for a in accepts) / len(accepts)


def acceptance_rate(accepts: Sequence[int], drafted: Sequence[int]) -> float:
    """alpha: accepted draft tokens over draft steps taken  [App. C.2]."""
    total = sum(drafted)
    return sum(accepts) / total if total else 0.0


def cost_coefficient(skip_ratio: float) -> float:
    """c = 1 - s  [App. C.2, text after Eq. (7)]."""
    return 1.0 - skip_ratio


def cost_coefficient_refined(s_mlp: float, s_attn: float, beta: float) -> float:
    """c = ((1 - s_mlp) + (1 - s_attn) * beta) / (1 + beta)  [App. C.2, Eq. (8)]."""
    return ((1.0 - s_mlp) + (1.0 - s_attn) * beta) / (1.0 + beta)


def expected_speedup(mean_len: float, alpha: float, c: float) -> float:
    """E(Spd.) = M*alpha / ((M - 1)*c + alpha)  [App. C.2, Eq. (7)]."""
    return mean_len * alpha / ((mean_len - 1.0) * c + alpha)
