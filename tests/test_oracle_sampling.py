"""Pins of the sampling oracle (``oracle/sampling.py``) against things other than itself (no GPU)."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from oracle import sampling as osamp


def test_temperature_and_nucleus_filter_match_the_library_warpers():
    """App. C.1 lists temperature and top_p as the standard generation settings of the transformer library the paper
    runs; the oracle's filtered distribution must be what that library's own logits warpers produce."""
    from transformers import TemperatureLogitsWarper, TopPLogitsWarper
    rng = np.random.default_rng(0)
    for trial in range(40):
        V = int(rng.integers(3, 400))
        logits = rng.standard_normal(V) * rng.uniform(0.3, 4.0)
        T, top_p = float(rng.choice([0.2, 0.7, 1.0, 1.5])), float(rng.choice([0.3, 0.85, 0.95]))
        if osamp.nucleus_margin(logits, T, top_p) < 1e-9:
            continue
        scores = torch.tensor(logits, dtype=torch.float64)[None]
        ids = torch.zeros((1, 1), dtype=torch.long)
        scores = TopPLogitsWarper(top_p=top_p, min_tokens_to_keep=1)(ids, TemperatureLogitsWarper(T)(ids, scores))
        want = torch.softmax(scores, dim=-1)[0].numpy()
        got = osamp.filtered_distribution(logits, T, top_p)
        assert np.array_equal(got > 0, want > 0)
        assert np.abs(got - want).max() < 1e-12


def test_filter_closed_forms():
    logits = np.log(np.array([1.0, 2.0, 3.0, 4.0]))
    assert np.allclose(osamp.filtered_distribution(logits, 1.0, 1.0), [0.1, 0.2, 0.3, 0.4], atol=1e-15)
    # mass before the 0.3 token is 0.4 < 0.65 (kept); before the 0.2 token it is 0.7 (dropped)
    assert np.allclose(osamp.filtered_distribution(logits, 1.0, 0.65), [0, 0, 3 / 7, 4 / 7], atol=1e-15)
    assert np.allclose(osamp.filtered_distribution(logits, 1.0, 0.4), [0, 0, 0, 1.0], atol=1e-15)     # 0.4 is not < 0.4: one token
    assert np.allclose(osamp.filtered_distribution(logits, 1.0, 1e-9), [0, 0, 0, 1.0], atol=1e-15)    # never empty
    # temperature sharpens: T = 0.5 squares the ratios
    assert np.allclose(osamp.filtered_distribution(logits, 0.5, 1.0), np.array([1, 4, 9, 16]) / 30.0, atol=1e-15)
    # equal probabilities: the lower id ranks first
    assert np.allclose(osamp.filtered_distribution(np.zeros(4), 1.0, 0.5), [0.5, 0.5, 0, 0], atol=1e-15)
    assert np.allclose(osamp.filtered_distribution(np.zeros(4), 1.0, 0.51), [1 / 3, 1 / 3, 1 / 3, 0], atol=1e-15)


def test_inverse_cdf_draw_matches_searchsorted():
    rng = np.random.default_rng(1)
    for trial in range(200):
        V = int(rng.integers(1, 60))
        w = rng.uniform(0, 1, V) * (rng.uniform(0, 1, V) < 0.6)
        if w.sum() == 0:
            w[int(rng.integers(0, V))] = 1.0
        u = float(rng.uniform(0, 1))
        cdf = np.cumsum(w)
        assert osamp.sample(w, u) == int(np.searchsorted(cdf, u * cdf[-1], side="right"))
    assert osamp.sample([0.0, 2.0, 0.0, 2.0], 0.0) == 1
    assert osamp.sample([0.0, 2.0, 0.0, 2.0], 0.4999) == 1
    assert osamp.sample([0.0, 2.0, 0.0, 2.0], 0.5) == 3
    assert osamp.sample([0.0, 2.0, 0.0, 2.0], 0.9999999) == 3


def test_low_temperature_reproduces_the_greedy_rule():
    """Temperature -> 0 puts all mass on the arg-max: drafting picks it whatever the uniform, and the keep / resample
    rule becomes the greedy one (keep while the draft equals the full model's arg-max, then emit that arg-max)."""
    rng = np.random.default_rng(2)
    for trial in range(50):
        V, k = 23, int(rng.integers(1, 6))
        pl, ql = rng.standard_normal((k + 1, V)), rng.standard_normal((k, V))
        for j in range(k):                      # make the draft agree on a random prefix
            if rng.uniform() < 0.7:
                ql[j] = pl[j] + 0.01 * rng.standard_normal(V)
        p = [osamp.filtered_distribution(x, 1e-7, 0.85) for x in pl]
        q = [osamp.filtered_distribution(x, 1e-7, 0.85) for x in ql]
        drafts = [osamp.sample(qj, float(rng.uniform())) for qj in q]
        assert drafts == [int(np.argmax(x)) for x in ql]
        got = osamp.accept_or_resample(p, q, drafts, rng.uniform(0, 1, k), float(rng.uniform()))
        assert got == oracle.accept(drafts, [int(np.argmax(x)) for x in pl])


def test_emitted_token_follows_the_full_models_distribution():
    """Losslessness of the sampled case (Sec. 1: the distribution of the generated tokens is unchanged): integrating
    over the three uniforms of a one-draft round (draw of the draft, keep test, final draw) the emitted token has
    exactly the full model's distribution p.  The probabilities are chosen so that every break point of the three
    inverse CDFs falls on a cell boundary of a 48-point midpoint grid, which makes the integration exact."""
    q = np.array([4, 4, 4, 2, 2]) / 16.0
    p = np.array([8, 2, 2, 4, 0]) / 16.0
    N = 48
    grid = (np.arange(N) + 0.5) / N
    emitted = np.zeros(5)
    kept = 0
    for ud in grid:
        d = osamp.sample(q, ud)
        for ua in grid:
            for uf in grid[::1]:
                a, nxt = osamp.accept_or_resample([p, p], [q], [d], [ua], uf)
                # the round emits the draft if it was kept, else the resampled token (the bonus token is not counted)
                emitted[d if a == 1 else nxt] += 1
                kept += a
    emitted /= N ** 3
    assert np.abs(emitted - p).max() < 1e-12
    assert abs(kept / N ** 3 - np.minimum(p, q).sum()) < 1e-12          # acceptance probability = overlap of p and q


def test_all_drafts_kept_when_the_models_agree_and_bonus_token_comes_from_p():
    rng = np.random.default_rng(3)
    V, k = 17, 4
    dist = [osamp.filtered_distribution(rng.standard_normal(V), 0.7, 0.9) for _ in range(k + 1)]
    drafts = [osamp.sample(dist[j], float(rng.uniform())) for j in range(k)]
    for uf in (0.0, 0.3, 0.77, 0.999):
        a, nxt = osamp.accept_or_resample(dist, dist[:k], drafts, rng.uniform(0, 1, k), uf)
        assert a == k and nxt == osamp.sample(dist[k], uf)
    # a draft the full model gives no mass is always rejected, and the replacement avoids tokens where q >= p
    p0 = np.array([0.5, 0.5, 0.0]); q0 = np.array([0.0, 0.5, 0.5])
    for ua, uf in itertools.product((0.0, 0.5, 0.99), (0.0, 0.5, 0.99)):
        assert osamp.accept_or_resample([p0, p0], [q0], [2], [ua], uf) == (0, 0)


def test_sampled_loop_is_the_greedy_loop_as_temperature_goes_to_zero():
    """With all mass on the arg-max the sampled draft-and-verify loop must emit the greedy loop's tokens and accept
    counts, whatever the uniforms (the greedy loop itself is pinned to plain greedy decoding elsewhere)."""
    import synthetic_inputs as si
    shape = si.SHAPES["tiny"]
    mask = si.skip_mask(0, 2 * shape.n_layers, 3)
    damp = {int(j): 0.02 for j in np.nonzero(mask)[0]}
    w = si.make_model_weights(shape, 0, gain_spread=0.1, damp=damp)
    prompt = si.uniform_tokens(0, 0, 12, shape.vocab).numpy()
    for k in (0, 2, 4):
        om = oracle.OracleModel(shape, w, 96)
        _, first, _ = om.prefill(prompt)
        want = om.generate(first, 20, k, mask)
        om2 = oracle.OracleModel(shape, w, 96)
        om2.prefill(prompt)
        got = osamp.generate_sampled(om2, first, 20, k, mask, 1e-7, 0.85, si.uniforms(k, 3, 19 * (2 * k + 1)))
        assert np.array_equal(got["tokens"], want["tokens"]) and np.array_equal(got["accepts"], want["accepts"])
        assert len(got["tokens"]) == 20
