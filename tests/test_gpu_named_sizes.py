"""The full-size workloads against token streams the CPU oracle wrote beforehand (``tests/golden/tokens_*.json``).

The oracle needs seconds per pass on 32 / 40 / 48-layer models, so its output is stored once by
``tests/golden/make_token_goldens.py`` (which calls only ``oracle/`` and ``synthetic_inputs/``); here the same seeded
inputs are rebuilt on the GPU from the recipe in each file and run through the C ABI as a user would: prompt pass,
cosine selection of the domain's mask, self-speculative decoding.  Exact: first token, selected domain and anchor,
every generated token, every round's accept count.  Within 2e-2: the pooled last hidden state and the logits of one
teacher-forced verification pass at the end of the prompt, on the entries the file samples.  Depth, width, prompt
length and draft length are the workloads' own; a file whose ``cut`` field is set generated fewer tokens than the
workload names (oracle time), nothing else.
"""
import glob
import json
import os

import numpy as np
import pytest
import torch

import synthetic_inputs as si

pytestmark = pytest.mark.gpu

HERE = os.path.dirname(os.path.abspath(__file__))
FILES = sorted(glob.glob(os.path.join(HERE, "golden", "tokens_*.json")),
               key=lambda p: (json.load(open(p))["shape"], json.load(open(p)).get("gamma", 1.0), p))
TOL = 2e-2

_weights = {}          # at most one model resident: (shape, seed, damp key) -> weights


@pytest.fixture(scope="module")
def kb():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding
    return binding


def _model_weights(shape, seed, damp):
    key = (shape.name, seed, tuple(sorted((damp or {}).items())))
    if key not in _weights:
        _weights.clear()
        torch.cuda.empty_cache()
        _weights[key] = si.make_model_weights(shape, seed, device="cuda", damp=damp)
    return _weights[key]


def _masks(rec, shape):
    seed, skip = rec["seed"], rec["skip"]
    if "pool" in rec:
        return si.nested_skip_masks(seed + 100, shape.n_layers, rec["n_domains"], rec["pool"][0], rec["pool"][1], skip[0], skip[1])[1]
    return np.stack([si.skip_mask_split(seed + 100 + i, shape.n_layers, skip[0], skip[1]) for i in range(rec["n_domains"])])


def _decode_following_the_oracle(sess, P, want_tokens, want_accepts, r, k, max_new):
    """Decodes max_new tokens and compares them with the oracle's.  Both sides' logits carry an error of up to TOL, so
    where the full model's two best logits are closer than 2 TOL the arg-max is not unique: at a first differing token
    the oracle's choice must be within 2 TOL of this side's best logit at that step (checked on the logits of a
    teacher-forced one-row pass), after which decoding continues from the oracle's token, so that every later token is
    still compared.  Returns the substitutions made: [(token index, logit gap)].  Accept counts are compared for the
    rounds before the first substitution (afterwards the rounds no longer line up).  The same holds for the DRAFT
    model's choices, which decide the accept counts but not the tokens: where the accept counts of a round differ
    although its tokens agree, the draft logits of that round's deciding step (recomputed here from the round's start)
    must have their two candidates within 2 TOL, and the rounds after it are compared by their tokens only.  Such a
    round is reported as (-(round index) - 1, gap) among the substitutions."""
    subs, start = [], 0
    first_run = True
    while start < max_new:
        got = sess.decode(max_new - start, k)
        seg = want_tokens[start:]
        bad = np.nonzero(got["tokens"] != seg)[0]
        if first_run:
            n_ok_rounds = len(want_accepts)
            if bad.size:                        # rounds that emitted only tokens before the first difference
                emitted, n_ok_rounds = 1, 0
                for a in want_accepts:
                    if emitted + a + 1 > bad[0]:
                        break
                    emitted += a + 1
                    n_ok_rounds += 1
            ga, wa = np.asarray(got["accepts"][:n_ok_rounds]), np.asarray(want_accepts[:n_ok_rounds])
            n_common = min(len(ga), len(wa))                    # equal unless a round was decided differently
            differ = np.nonzero(ga[:n_common] != wa[:n_common])[0]
            assert differ.size or len(ga) == len(wa)
            if differ.size:
                rd = int(differ[0])
                emitted = 1 + int(np.sum(wa[:rd] + 1))          # tokens out when round rd starts
                a_min = int(min(ga[rd], wa[rd]))                # drafts both sides kept; step a_min decided differently
                t_true = int(want_tokens[emitted + a_min])      # the full model's token there (both sides emitted it)
                sess.set_length(P + emitted - 1)
                sess.set_pending(int(want_tokens[emitted - 1]))
                _, dl = sess.draft(k, want_logits=True)
                top = torch.topk(dl[a_min], 2)
                gap = float(top.values[0] - dl[a_min][t_true]) if int(top.indices[0]) != t_true else float(top.values[0] - top.values[1])
                assert gap < 2 * TOL, f"round {rd}: accept counts {ga[rd]} / {wa[rd]} differ and the draft's choice is no near-tie ({gap})"
                subs.append((-rd - 1, gap))
            if not bad.size and not differ.size:
                st = got["stats"]
                assert (st["rounds"], st["drafted"], st["accepted"]) == (r["rounds"], r["drafted"], r["accepted"])
            first_run = False
        if not bad.size:
            break
        i = start + int(bad[0])                 # token i differs; tokens before it agree, so their K/V rows are valid
        assert i >= 1
        sess.set_length(P + i - 1)
        sess.set_pending(int(want_tokens[i - 1]))
        g = sess.verify([], want_logits=True)   # the full model's logits for token i, given the oracle's prefix
        lg = g["logits"][0]
        gap = float(lg.max() - lg[int(want_tokens[i])])
        assert gap < 2 * TOL, f"token {i}: the oracle's token is {gap} below this side's best logit - not a near-tie"
        subs.append((i, gap))
        sess.set_pending(int(want_tokens[i]))   # follow the oracle
        start = i
    return subs


def test_golden_files_are_present():
    assert FILES, "no tests/golden/tokens_*.json"


@pytest.mark.parametrize("path", FILES, ids=[os.path.basename(p)[7:-5] for p in FILES])
def test_workload_matches_the_oracles_stored_output(kb, path):
    rec = json.load(open(path))
    shape = si.SHAPES[rec["shape"]]
    seed, k, max_new = rec["seed"], rec["k"], rec["max_new"]
    nd, per = rec["n_domains"], rec["anchors_per_domain"]
    masks = _masks(rec, shape)
    damp = None
    if "gamma" in rec:
        damp = {int(j): rec["gamma"] for j in np.nonzero(masks[rec["shaped_domain"]])[0]}
    w = _model_weights(shape, seed, damp)
    anchors = si.anchors(seed, nd, per, shape.d_model, rec["sigma_a"]).cuda()
    stream = "requests_per_domain" in rec
    if stream:
        labels = si.request_stream(seed, nd, rec["requests_per_domain"], rec["mix_ratio"])
        lengths = si.prompt_lengths(seed, nd * rec["requests_per_domain"], *rec["prompt_range"])
        cen = si.domain_centroids(seed, nd, shape.d_model).cuda()
    max_seq = max(r["prompt_len"] for r in rec["requests"]) + max_new + 64
    sess = kb.Session.from_shape(shape, w, max_seq, max_draft=max(k, 8), anchors=anchors, skip_masks=masks,
                                 anchors_per_domain=per)
    worst_logit, worst_pooled = 0.0, 0.0
    near_ties = []
    for r in rec["requests"]:
        P = r["prompt_len"]
        if stream:
            i = r["index"]
            assert labels[i] == r["label"] and lengths[i] == P
            prompt = si.uniform_tokens(seed, 1 + i, P, shape.vocab).numpy()
        else:
            prompt = si.uniform_tokens(seed, 0, P, shape.vocab).numpy()
        first, pooled = sess.prefill(prompt, want_pooled=True)
        assert first == r["first_token"], f"first token; oracle margin {r['first_margin']}"
        pg = pooled[torch.tensor(r["pooled_index"], device="cuda")].cpu().numpy()
        worst_pooled = max(worst_pooled, float(np.abs(pg - np.array(r["pooled"], dtype=np.float32)).max()))
        assert worst_pooled < TOL
        if stream:
            c = cen[r["label"]]
            query = (pooled + 4.0 * pooled.norm() / c.norm() * c).contiguous()   # a draw from the domain's cluster
            dom, anc, cos = sess.select_skipset(query)
            assert dom == r["label"]
        else:
            dom, anc, cos = sess.select_skipset()
        assert (dom, anc) == (r["domain"], r["anchor"]), f"selection; oracle gap between domains {r['domain_gap']}"
        assert abs(cos - r["cosine"]) < 1e-4
        if "explicit_mask_domain" in rec:
            sess.set_skipmask(masks[rec["explicit_mask_domain"]])
        want_tokens, want_accepts = np.array(r["tokens"], np.int32), np.array(r["accepts"], np.int32)
        subs = _decode_following_the_oracle(sess, P, want_tokens, want_accepts, r, k, max_new)
        near_ties.extend(subs)
        # one teacher-forced verification pass at the prompt's end: sampled logits of every row
        sess.set_length(P)
        sess.set_pending(first)
        rows = r["verify_rows"]
        assert rows[0] == first
        g = sess.verify(rows[1:], want_logits=True)
        lg = g["logits"][:, torch.tensor(r["logit_index"], device="cuda")].cpu().numpy()
        worst_logit = max(worst_logit, float(np.abs(lg - np.array(r["logits"], dtype=np.float32)).max()))
        assert worst_logit < TOL
        n_acc = 0
        while n_acc < len(rows) - 1 and r["verify_argmax"][n_acc] == rows[n_acc + 1]:
            n_acc += 1
        assert (g["n_accepted"], g["next_token"]) == (n_acc, r["verify_argmax"][n_acc])
    sess.close()
    n_tok = sum(len(r["tokens"]) for r in rec["requests"])
    print(f"\n[{rec['case']}] {n_tok} tokens, {len(near_ties)} near-tie substitution(s) {[(i, round(g, 5)) for i, g in near_ties]}; "
          f"max |logit - oracle| on sampled entries {worst_logit:.3e}, pooled {worst_pooled:.3e}, "
          f"oracle min margin {min(r['min_margin'] for r in rec['requests']):.3e}")
    assert len([t for t in near_ties if t[0] >= 0]) <= max(3, n_tok // 16)
