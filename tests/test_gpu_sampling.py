"""Sampling operators (temperature / top-p filtering, inverse-CDF draw, keep-or-resample round) against the CPU oracle
on the same logits and the same uniforms.  Probabilities within 1e-6; sets of kept tokens, drawn tokens and accept
counts exact wherever the oracle's decision is not within rounding of flipping (the oracle reports that margin: a draw
that lands within 1e-5 of a CDF step, or a nucleus boundary within 1e-5 of top_p, is a coin toss between fp32 and fp64
and is skipped, and the test checks that such cases stay rare)."""
import numpy as np
import pytest
import torch

import synthetic_inputs as si
from oracle import sampling as osamp

pytestmark = pytest.mark.gpu
MARGIN = 2e-6            # draws: distance of u from the nearest CDF step (fp32 running sums of <= 152 k terms)
NUCLEUS_MARGIN = 2e-6    # nucleus: distance of the mass ranked before a token from top_p


@pytest.fixture(scope="module")
def kb():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding
    return binding


def _logits(seed, rows, V, spread):
    return (si.normal_f32(seed, 900, torch.arange(rows * V), 1.0).view(rows, V) * spread).contiguous()


@pytest.mark.parametrize("V,spread", [(5, 1.0), (1000, 1.4), (1024, 0.3), (3001, 1.4), (32000, 1.4), (152064, 1.4)])
@pytest.mark.parametrize("T,top_p", [(0.2, 0.85), (1.0, 0.85), (0.7, 1.0), (1.0, 2.0), (0.2, 1e-4)])
def test_filtered_probs_match_oracle(kb, V, spread, T, top_p):
    rows = 3 if V > 40000 else 5
    lg = _logits(V + int(10 * T), rows, V, spread)
    got = kb.knnssd_filtered_probs(lg.cuda(), T, top_p).cpu().numpy()
    clear = 0
    for r in range(rows):
        want = osamp.filtered_distribution(lg[r].numpy(), T, top_p)
        differ = (got[r] > 0) != (want > 0)
        assert abs(got[r].sum() - 1.0) < 1e-5
        if osamp.nucleus_margin(lg[r].numpy(), T, top_p) >= NUCLEUS_MARGIN or top_p > 1.0:
            clear += 1
            assert not differ.any(), f"row {r}: kept sets differ"
            assert np.abs(got[r] - want).max() < 1e-6
        else:
            # the mass ranked before some token is within fp32 rounding of top_p (always so for flat distributions over
            # a large vocabulary, or top_p = 1): those tokens' kept / dropped decisions are coin tosses.  Only tokens at
            # that boundary may differ - each no more probable than the least probable kept token allows - and the
            # rest agrees up to the renormalisation by their mass
            edge = max(want[differ].max(initial=0.0), float(got[r][differ].max(initial=0.0)))
            kept_min = want[want > 0].min()
            assert edge <= 4 * kept_min + 1e-7
            assert np.abs(got[r] - want).max() < 1e-6 + 1.5 * max(edge, differ.sum() * edge * want.max())
    assert clear >= 1 or T >= 0.7


def test_equal_logits_rank_by_id(kb):
    lg = torch.zeros((1, 4096)).cuda()
    got = kb.knnssd_filtered_probs(lg, 1.0, 0.25).cpu().numpy()[0]
    want = osamp.filtered_distribution(np.zeros(4096), 1.0, 0.25)
    # 4096 equal probabilities of 2**-12: exactly the first 1024 ids reach 0.25 (exact in fp32 and fp64 alike)
    assert np.array_equal(got > 0, want > 0) and (got > 0).sum() == 1024 and (got[:1024] > 0).all()
    assert np.abs(got - want).max() < 1e-9
    two = torch.tensor([[0.0, 3.0, 3.0, -1.0]]).cuda()            # two tokens tie at the top: the lower id alone is kept
    assert np.array_equal(kb.knnssd_filtered_probs(two, 1.0, 0.3).cpu().numpy()[0] > 0, [False, True, False, False])


@pytest.mark.parametrize("V", [7, 1000, 32000, 152064])
def test_inverse_cdf_draw_matches_oracle(kb, V):
    lg = _logits(V, 2, V, 1.4)
    probs = kb.knnssd_filtered_probs(lg.cuda(), 0.2, 0.85)
    wide = kb.knnssd_filtered_probs(lg.cuda(), 1.0, 2.0)
    us = si.uniforms(V, 1, 24)
    skipped = 0
    for dist in (probs[0], wide[1]):
        w = dist.cpu().numpy().astype(np.float64)
        for u in list(us) + [0.0, 0.99999994]:
            if osamp.sample_gap(w, u) < MARGIN:
                skipped += 1
                continue
            assert kb.knnssd_sample_token(dist.contiguous(), u) == osamp.sample(w, u)
    assert skipped <= 26
    sparse = torch.zeros(V); sparse[V // 2] = 2.0; sparse[V - 1] = 2.0
    assert kb.knnssd_sample_token(sparse.cuda(), 0.25) == V // 2
    assert kb.knnssd_sample_token(sparse.cuda(), 0.75) == V - 1


@pytest.mark.parametrize("V,k", [(11, 1), (1000, 4), (32000, 4), (32000, 8), (152064, 2)])
def test_keep_or_resample_round_matches_oracle(kb, V, k):
    """Draft logits close to the full model's (so that keep and reject both occur), drafts drawn from q with seeded
    uniforms, then the round on both sides with the same uniforms."""
    checked, kept_total, rejected_rounds = 0, 0, 0
    for trial in range(6):
        pl = _logits(100 * trial + k, k + 1, V, 1.4)
        noise = _logits(100 * trial + k + 50, k, V, 1.0 if trial % 2 else 0.05)
        ql = pl[:k] + noise
        T, top_p = (0.2, 0.85) if trial % 3 else (1.0, 0.95)
        p_dev = kb.knnssd_filtered_probs(pl.cuda(), T, top_p)
        q_dev = kb.knnssd_filtered_probs(ql.cuda(), T, top_p)
        p = p_dev.cpu().numpy().astype(np.float64)
        q = q_dev.cpu().numpy().astype(np.float64)
        us = si.uniforms(trial, 7 + k, 2 * k + 1)
        drafts = [osamp.sample(q[j], us[j]) for j in range(k)]
        ua, uf = us[k:2 * k], us[2 * k]
        want = osamp.accept_or_resample(p, q, drafts, ua, uf)
        # the oracle here works on the SAME fp32 distributions, so only the keep test and the final draw can round apart
        a = want[0]
        resid = np.maximum(p[a] - q[a], 0.0) if a < k else p[k]
        if osamp.accept_margin(p, q, drafts, ua) < 1e-7 or osamp.sample_gap(resid if resid.sum() > 0 else p[a], uf) < MARGIN:
            continue
        got = kb.knnssd_spec_accept(p_dev, q_dev, drafts, ua, uf)
        assert got == want
        checked += 1
        kept_total += a
        rejected_rounds += int(a < k)
    assert checked >= 4 and kept_total >= 1 and (rejected_rounds >= 1 or k == 1)


def test_round_without_drafts_and_bad_arguments(kb):
    lg = _logits(1, 1, 500, 1.4)
    p = kb.knnssd_filtered_probs(lg.cuda(), 0.7, 0.9)
    a, nxt = kb.knnssd_spec_accept(p, None, [], [], 0.5)
    assert a == 0 and nxt == osamp.sample(p[0].cpu().numpy().astype(np.float64), 0.5)
    E = kb.KnnssdError
    with pytest.raises(E) as e:
        kb.knnssd_filtered_probs(lg.cuda(), 0.0, 0.9)
    assert e.value.status == 1
    with pytest.raises(E) as e:
        kb.knnssd_sample_token(p[0].contiguous(), 1.0)
    assert e.value.status == 1
    with pytest.raises(E) as e:
        kb.knnssd_spec_accept(torch.cat([p, p]), p, [500], [0.5], 0.5)          # draft outside the vocabulary
    assert e.value.status == 1


# ---- the sampled draft-and-verify loop ------------------------------------------------------------------------------

def _to_dev(w):
    return {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}


@pytest.mark.parametrize("shape_name", ["tiny", "stream-bf16"])
def test_sampled_loop_at_vanishing_temperature_is_the_greedy_loop(kb, shape_name):
    shape = si.SHAPES[shape_name]
    mask = si.skip_mask(0, 2 * shape.n_layers, 3)
    damp = {int(j): 0.05 for j in np.nonzero(mask)[0]}
    w = _to_dev(si.make_model_weights(shape, 0, damp=damp, gain_spread=0.1))
    sess = kb.Session.from_shape(shape, w, 160, max_draft=8)
    sess.set_skipmask(mask)
    prompt = si.uniform_tokens(0, 0, 33, shape.vocab).numpy()
    for k in (0, 3, 8):
        first = sess.prefill(prompt)
        want = sess.decode(24, k)
        assert sess.prefill(prompt) == first
        got = sess.decode_sampled(24, k, 1e-6, 0.85, si.uniforms(k, 5, 23 * (2 * k + 1)))
        assert np.array_equal(got["tokens"], want["tokens"]) and np.array_equal(got["accepts"], want["accepts"])
        assert got["stats"]["accepted"] == want["stats"]["accepted"]


@pytest.mark.parametrize("shape_name,T,need", [("tiny", 0.5, 1e-4), ("stream-bf16", 0.05, 2e-2)])
def test_sampled_loop_matches_oracle_on_a_run_with_clear_decisions(kb, shape_name, T, need):
    """Same uniforms on both sides.  A draw within rounding of a CDF step is a coin toss between the two sides' slightly
    different logits, so the oracle reports how close any decision of a run came to flipping and the first seeded
    streams of uniforms whose runs stay clear of that are the ones compared.  top_p = 2 keeps every token: over a
    thousand tokens some nucleus boundary always lies within rounding of top_p (the filter has its own parity test
    above).  The fp32 model (logits equal to ~1e-5) is compared at temperature 0.5; the bf16 one, whose logits differ
    by a few 1e-4 between the sides, at a temperature low enough that the CDF's steps are far larger than that."""
    import oracle
    from oracle import sampling as osamp
    shape = si.SHAPES[shape_name]
    mask = si.skip_mask(0, 2 * shape.n_layers, 3)
    damp = {int(j): 0.05 for j in np.nonzero(mask)[0]}
    w = si.make_model_weights(shape, 0, damp=damp, gain_spread=0.1)
    prompt = si.uniform_tokens(0, 0, 21, shape.vocab).numpy()
    k, max_new, top_p = 3, 14, 2.0
    sess = kb.Session.from_shape(shape, _to_dev(w), 96, max_draft=4)
    sess.set_skipmask(mask)
    compared = 0
    for stream in range(80):
        us = si.uniforms(11, 100 + stream, (max_new - 1) * (2 * k + 1))
        om = oracle.OracleModel(shape, w, 96)
        _, first, _ = om.prefill(prompt)
        want = osamp.generate_sampled(om, first, max_new, k, mask, T, top_p, us)
        if want["margin"] < need:
            continue
        assert sess.prefill(prompt) == first
        got = sess.decode_sampled(max_new, k, T, top_p, us)
        assert np.array_equal(got["tokens"], want["tokens"]), f"stream {stream}, oracle margin {want['margin']}"
        assert np.array_equal(got["accepts"], want["accepts"])
        compared += 1
        if compared == 3:
            break
    assert compared >= 1, "no stream of uniforms gave a run clear of near-ties"


def test_sampled_loop_rejects_bad_arguments(kb):
    shape = si.SHAPES["tiny"]
    sess = kb.Session.from_shape(shape, _to_dev(si.make_model_weights(shape, 0)), 64, max_draft=4)
    prompt = si.uniform_tokens(0, 0, 10, shape.vocab).numpy()
    E = kb.KnnssdError
    with pytest.raises(E) as e:
        sess.decode_sampled(8, 2, 0.5, 0.9, si.uniforms(0, 0, 35))         # before prefill
    assert e.value.status == 4
    sess.prefill(prompt)
    sess.set_skipmask(np.zeros(8, np.uint8))
    with pytest.raises(E) as e:
        sess.decode_sampled(8, 2, 0.5, 0.9, si.uniforms(0, 0, 34))         # one uniform short
    assert e.value.status == 1
    with pytest.raises(E) as e:
        sess.decode_sampled(8, 2, 0.0, 0.9, si.uniforms(0, 0, 35))
    assert e.value.status == 1
    bad = si.uniforms(0, 0, 35); bad[3] = 1.0
    with pytest.raises(E) as e:
        sess.decode_sampled(8, 2, 0.5, 0.9, bad)
    assert e.value.status == 1
    got = sess.decode_sampled(8, 2, 0.5, 0.9, si.uniforms(0, 0, 35))
    assert len(got["tokens"]) == 8 and (got["tokens"] >= 0).all() and (got["tokens"] < shape.vocab).all()
