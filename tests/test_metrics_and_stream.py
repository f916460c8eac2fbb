"""Host-side reporting formulas against the numbers the paper prints, and the
request-stream generator against the mix-ratio law (no GPU)."""
import os
from collections import Counter

import pytest

import synthetic_inputs as si
from paper_2505_16162_b200 import metrics


def _golden():
    out = {}
    with open(os.path.join(os.path.dirname(__file__), "golden", "paper_metric_examples.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                name, value = line.split()[:2]
                out[name] = float(value)
    return out


def test_cost_coefficients_match_the_printed_example():
    g = _golden()
    assert metrics.cost_coefficient(0.45) == pytest.approx(g["c_plain_s045"], abs=1e-12)
    assert round(metrics.cost_coefficient_refined(0.42, 0.48, 2.3), 3) == g["c_refined_b23"]
    # beta = 1 reduces the refined form to 1 - s when both ratios equal s
    assert metrics.cost_coefficient_refined(0.45, 0.45, 1.0) == pytest.approx(0.55, abs=1e-12)


def test_expected_speedup_reproduces_the_table_row():
    g = _golden()
    e = metrics.expected_speedup(g["table_M"], g["table_alpha"], metrics.cost_coefficient(0.45))
    assert round(e, 2) == g["table_speedup"]
    # a draft model that costs as much as the target and is always right gains nothing beyond M*alpha/(M-1+alpha)
    assert metrics.expected_speedup(1.0, 1.0, 1.0) == pytest.approx(1.0)


def test_length_and_acceptance_definitions():
    accepts, drafted = [4, 0, 2, 1], [4, 4, 4, 1]
    assert metrics.mean_generated_length(accepts) == pytest.approx((5 + 1 + 3 + 2) / 4)
    assert metrics.acceptance_rate(accepts, drafted) == pytest.approx(7 / 13)


@pytest.mark.parametrize("r", [0.0, 0.3, 0.7, 1.0])
def test_stream_follows_the_mix_ratio_law(r):
    n_dom, per = 5, 2000
    s = si.request_stream(11, n_dom, per, r)
    assert Counter(s) == {d: per for d in range(n_dom)}
    # look only at the first half, before quotas start to bind
    half = s[: len(s) // 2]
    switches = sum(a != b for a, b in zip(half, half[1:]))
    frac = switches / (len(half) - 1)
    if r == 0.0:
        assert switches == 0 or all(half[i] == half[i + 1] or half[: i + 1].count(half[i]) == per
                                    for i in range(len(half) - 1))
    elif r == 1.0:
        assert frac == 1.0
    else:
        assert abs(frac - r) < 0.03
        moves = Counter((a, b) for a, b in zip(half, half[1:]) if a != b)
        for a in range(n_dom):
            tot = sum(v for (x, _), v in moves.items() if x == a)
            for b in range(n_dom):
                if b != a and tot > 50:
                    assert abs(moves[(a, b)] / tot - 1 / (n_dom - 1)) < 0.1


def test_stream_with_r0_is_task_by_task():
    s = si.request_stream(0, 5, 40, 0.0)
    runs = [s[i] for i in range(len(s)) if i == 0 or s[i] != s[i - 1]]
    assert len(runs) == 5 and len(set(runs)) == 5


def test_generators_are_device_independent_bits():
    import torch
    a = si.normal_weight(3, 99, 7, 33, 0.02, "bf16")
    b = si.normal_weight(3, 99, 7, 33, 0.02, "fp32").to(torch.bfloat16)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    assert si.hash_u64_int(5, 9, 1234) == int(si.hash_u64(5, 9, torch.tensor([1234])).item()) % (1 << 64)
    assert abs(float(si.normal_weight(0, 1, 512, 512, 0.02, "fp32").std()) - 0.02) < 2e-4
    assert si.skip_mask_split(0, 40, 19, 17)[0::2].sum() == 19 and si.skip_mask_split(0, 40, 19, 17)[1::2].sum() == 17
