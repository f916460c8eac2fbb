"""CUDA path against the CPU oracle, element by element on the same seeded inputs.

Everything goes through the C ABI (via the thin binding).  Exact for tokens, accept counts and
selected domain / anchor; max-abs tolerance for logits and hidden states: 1e-4 for the fp32
configuration, 2e-2 for bf16 weights (both sides accumulate in >= fp32 and round K/V to bf16).
"""
import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as si

pytestmark = pytest.mark.gpu

TOL = {"fp32": 1e-4, "bf16": 2e-2}


@pytest.fixture(scope="module")
def kb():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding
    return binding


def _to_dev(w):
    return {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}


def _pair(kb, shape_name, seed=0, max_seq=160, gain_spread=0.1, damp=None, anchors=None, masks=None, per=0,
          n_layers=None, max_draft=8, pool_mode=0):
    shape = si.SHAPES[shape_name]
    if n_layers:
        shape = shape.with_layers(n_layers)
    w = si.make_model_weights(shape, seed, gain_spread=gain_spread, damp=damp)
    om = oracle.OracleModel(shape, w, max_seq)
    sess = kb.Session.from_shape(shape, _to_dev(w), max_seq, max_draft=max_draft,
                                 anchors=None if anchors is None else anchors.cuda(), skip_masks=masks,
                                 anchors_per_domain=per, pool_mode=pool_mode)
    return shape, om, sess


# ---- per-kernel: weight-streaming linear ----------------------------------------------------------

@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("n_out,n_in,M", [(1, 8, 1), (37, 72, 3), (1003, 328, 1), (1003, 328, 5), (2051, 1384, 9),
                                          (515, 2056, 16), (4099, 512, 2), (300, 5120, 7),
                                          # streaming-kernel shapes (bf16, n_in % 128 == 0, M <= 8): one and several
                                          # batches per CTA, partial last column tile, fewer rows than CTAs
                                          (20011, 256, 3), (5120, 5120, 5), (333, 13824, 8), (4099, 1152, 1),
                                          (160, 1024, 8), (7, 2048, 2), (40000, 384, 1)])
def test_linear_matches_oracle(kb, dtype, n_out, n_in, M):
    W = si.normal_weight(1, 77, n_out, n_in, 0.02, dtype)
    x = si.normal_f32(2, 78, torch.arange(M * n_in), 1.0).view(M, n_in).contiguous()
    want = oracle.linear(W, x.numpy())
    got = kb.knnssd_linear(W.cuda(), x.cuda()).cpu().numpy()
    assert np.abs(got - want).max() < 2e-5 * max(1.0, np.abs(want).max())


def test_linear_rows_do_not_depend_on_batch(kb):
    """A row of an M-row launch is bit-identical to the same row launched alone."""
    for n_in, top in ((1384, 9), (1152, 8)):          # generic kernel; streaming kernel
        W = si.normal_weight(1, 77, 1003, n_in, 0.02, "bf16").cuda()
        x = si.normal_f32(2, 78, torch.arange(top * n_in), 1.0).view(top, n_in).contiguous().cuda()
        full = kb.knnssd_linear(W, x)
        for M in (1, 2, 5):
            assert torch.equal(kb.knnssd_linear(W, x[:M].contiguous()), full[:M])
        assert torch.equal(kb.knnssd_linear(W, x[4:5].contiguous())[0], full[4])


def test_linear_rejects_bad_arguments(kb):
    W = torch.zeros((4, 12), device="cuda")
    x = torch.zeros((1, 12), device="cuda")
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_linear(W, x)          # n_in not a multiple of 8
    assert e.value.status == 2


# ---- per-kernel: cosine top-1 -----------------------------------------------------------------------

def test_cosine_top1_matches_oracle(kb):
    rng = np.random.default_rng(5)
    for trial in range(30):
        nd, per, d = int(rng.integers(1, 7)), int(rng.integers(1, 12)), int(rng.integers(1, 700))
        a = (rng.standard_normal((nd * per, d)) * rng.uniform(0.1, 10, (nd * per, 1))).astype(np.float32)
        v = rng.standard_normal(d).astype(np.float32)
        dom, anc, cs = oracle.knn_select(v, a, nd, per)
        best, cos = kb.knnssd_cosine_top1(torch.tensor(v).cuda(), torch.tensor(a).cuda())
        assert best == dom * per + anc
        assert abs(cos - cs) < 1e-5
    a = si.anchors(0, 5, 10, 5120, 0.2)
    best, cos = kb.knnssd_cosine_top1((2.5 * a[17]).cuda(), a.cuda())
    assert best == 17 and abs(cos - 1.0) < 1e-5
    dup = torch.cat([a[:3], a[:3]]).cuda()
    assert kb.knnssd_cosine_top1(a[1].cuda(), dup)[0] == 1           # tie -> lowest index
    for bad_q, bad_a in [(torch.zeros(5120), a), (a[0], torch.cat([a[:4], torch.zeros(1, 5120)]))]:
        with pytest.raises(kb.KnnssdError) as e:
            kb.knnssd_cosine_top1(bad_q.cuda(), bad_a.contiguous().cuda())
        assert e.value.status == 5


# ---- whole path on small shapes -------------------------------------------------------------------

CASES = [("tiny", 32, 32), ("gqa-fp32", 21, 19), ("ragged-bf16", 33, 24), ("gqa-bf16", 40, 24),
         ("stream-bf16", 37, 24)]


@pytest.mark.parametrize("shape_name,prompt_len,max_new", CASES)
def test_prefill_pool_select_match_oracle(kb, shape_name, prompt_len, max_new):
    base = si.SHAPES[shape_name]
    nd, per = 3, 8
    anchors = si.anchors(0, nd, per, base.d_model, 0.5, clustered=False)
    masks = np.stack([si.skip_mask(s, 2 * base.n_layers, 3) for s in range(nd)])
    shape, om, sess = _pair(kb, shape_name, anchors=anchors, masks=masks, per=per)
    prompt = si.uniform_tokens(0, 0, prompt_len, shape.vocab).numpy()
    pooled_o, first_o, _ = om.prefill(prompt)
    first_g, pooled_g = sess.prefill(prompt, want_pooled=True)
    assert first_g == first_o
    assert np.abs(pooled_g.cpu().numpy() - pooled_o).max() < TOL[shape.dtype]
    dom_o, anc_o, cos_o = oracle.knn_select(pooled_o, anchors.numpy(), nd, per)
    dom_g, anc_g, cos_g = sess.select_skipset()
    assert (dom_g, anc_g) == (dom_o, anc_o) and abs(cos_g - cos_o) < 1e-4
    # the selected domain's mask is now active: drafting must follow it
    d_g = sess.draft(3)
    cur, want = first_o, []
    for j in range(3):
        cur = int(om.forward([cur], prompt_len + j, skip_mask=masks[dom_o], want_logits=False)["argmax"][0])
        want.append(cur)
    assert list(d_g) == want


@pytest.mark.parametrize("shape_name,prompt_len,max_new", CASES)
def test_teacher_forced_logits_and_hidden_match_oracle(kb, shape_name, prompt_len, max_new):
    shape, om, sess = _pair(kb, shape_name)
    mask = si.skip_mask(0, 2 * shape.n_layers, 3 if shape.n_layers > 2 else 2)
    prompt = si.uniform_tokens(0, 0, prompt_len, shape.vocab).numpy()
    _, first_o, _ = om.prefill(prompt)
    assert sess.prefill(prompt) == first_o
    sess.set_skipmask(mask)
    tol = TOL[shape.dtype]
    n = prompt_len
    forced = si.uniform_tokens(9, 1, 40, shape.vocab).numpy()     # an arbitrary token stream both sides follow
    pending, fi = first_o, 0
    for k in (4, 1, 8, 2, 0):
        # draft logits under the mask, step by step (the oracle is fed the GPU's own chain only if it agrees)
        if k:
            d_tokens, d_logits = sess.draft(k, want_logits=True)
            cur = pending
            for j in range(k):
                o = om.forward([cur], n + j, skip_mask=mask)
                assert np.abs(d_logits[j].cpu().numpy() - o["logits"][0]).max() < tol
                assert int(o["argmax"][0]) == int(d_tokens[j])
                cur = int(o["argmax"][0])
        rows = forced[fi:fi + k]
        fi += k
        o = om.forward(np.concatenate([[pending], rows]).astype(np.int32), n, want_hidden=True)
        g = sess.verify(rows, want_logits=True, want_hidden=True)
        assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < tol
        assert np.abs(g["hidden"].cpu().numpy() - o["hidden"]).max() < tol
        a, nxt = oracle.accept(rows, o["argmax"])
        assert (g["n_accepted"], g["next_token"]) == (a, nxt)
        n += a + 1
        om.length = n
        assert sess.length == n
        pending = nxt


@pytest.mark.parametrize("k", [1, 2, 4, 8])
@pytest.mark.parametrize("shape_name,prompt_len,max_new", CASES)
def test_generate_matches_oracle_exactly(kb, shape_name, prompt_len, max_new, k):
    base = si.SHAPES[shape_name]
    mask = si.skip_mask(0, 2 * base.n_layers, 3 if base.n_layers > 2 else 2)
    damp = {int(j): 0.05 for j in np.nonzero(mask)[0]}          # so that accept counts span 0..k
    shape, om, sess = _pair(kb, shape_name, damp=damp)
    prompt = si.uniform_tokens(0, 0, prompt_len, shape.vocab).numpy()
    _, first, _ = om.prefill(prompt)
    want = om.generate(first, max_new, k, mask)
    sess.set_skipmask(mask)
    got = sess.generate(prompt, max_new, k)
    assert np.array_equal(got["tokens"], want["tokens"]), f"oracle min margin {want['min_margin']}"
    assert np.array_equal(got["accepts"], want["accepts"])
    st = got["stats"]
    assert (st["rounds"], st["drafted"], st["accepted"], st["tokens"]) == \
           (want["rounds"], want["drafted"], want["accepted"], max_new)
    # losslessness on the GPU itself: k = 0 is plain greedy decoding with the full model
    plain = sess.generate(prompt, max_new, 0)
    assert np.array_equal(plain["tokens"], got["tokens"])


def test_full_width_13b_layers_match_oracle(kb):
    """The widths of the LLaMA-2-13B-shaped workload (d 5120, 40 heads, FFN 13824, vocab 32000) on two layers, so that the
    oracle finishes in seconds: the launch configuration the benchmark times (persistent pass kernel, 148 CTAs), a
    prompt that spans several 64-position attention segments with a ragged tail, k = 4 and k = 8."""
    shape = si.SHAPES["llama13b"].with_layers(2)
    mask = np.array([1, 0, 0, 1], np.uint8)                    # skip attention of layer 0 and MLP of layer 1
    damp = {0: 0.02, 3: 0.02}
    w = si.make_model_weights(shape, 5, device="cuda", damp=damp, gain_spread=0.1)
    wc = {k: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for k, v in w.items()}
    om = oracle.OracleModel(shape, wc, 224)
    sess = kb.Session.from_shape(shape, w, 224, max_draft=8)
    prompt = si.uniform_tokens(7, 0, 150, shape.vocab).numpy()
    pooled_o, first_o, _ = om.prefill(prompt)
    first_g, pooled_g = sess.prefill(prompt, want_pooled=True)
    assert first_g == first_o
    assert np.abs(pooled_g.cpu().numpy() - pooled_o).max() < TOL["bf16"]
    # teacher-forced rows: logits and hidden states of one verification pass
    rows = si.uniform_tokens(8, 1, 4, shape.vocab).numpy()
    o = om.forward(np.concatenate([[first_o], rows]).astype(np.int32), 150, want_hidden=True)
    g = sess.verify(rows, want_logits=True, want_hidden=True)
    assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < TOL["bf16"]
    assert np.abs(g["hidden"].cpu().numpy() - o["hidden"]).max() < TOL["bf16"]
    assert (g["n_accepted"], g["next_token"]) == oracle.accept(rows, o["argmax"])
    for k in (4, 8):
        om.length = 150
        sess.set_length(150)
        sess.set_pending(first_o)
        sess.set_skipmask(mask)
        want = om.generate(first_o, 14, k, mask)
        got = sess.decode(14, k)
        assert np.array_equal(got["tokens"], want["tokens"]), f"k={k}: oracle min margin {want['min_margin']}"
        assert np.array_equal(got["accepts"], want["accepts"])


@pytest.mark.parametrize("shape_name,prompt_len", [("qwen14b", 186), ("llama7b", 120)])
def test_full_width_other_shapes_match_oracle(kb, shape_name, prompt_len):
    """Full widths of the Qwen-2.5-14B-shaped (GQA 40/8, vocab 152064, theta 1e6) and LLaMA-2-7B-shaped workloads on two
    layers; the Qwen case starts six positions before a 64-position segment boundary, so drafted and verified rows
    straddle it."""
    shape = si.SHAPES[shape_name].with_layers(2)
    mask = np.array([0, 1, 1, 0], np.uint8)                    # skip MLP of layer 0 and attention of layer 1
    damp = {1: 0.02, 2: 0.02}
    w = si.make_model_weights(shape, 6, device="cuda", damp=damp, gain_spread=0.1)
    wc = {k: ([t.cpu() for t in v] if isinstance(v, list) else v.cpu()) for k, v in w.items()}
    om = oracle.OracleModel(shape, wc, prompt_len + 40)
    sess = kb.Session.from_shape(shape, w, prompt_len + 40, max_draft=8)
    prompt = si.uniform_tokens(11, 0, prompt_len, shape.vocab).numpy()
    _, first_o, _ = om.prefill(prompt)
    assert sess.prefill(prompt) == first_o
    sess.set_skipmask(mask)
    for k in (4, 8):
        om.length = prompt_len
        sess.set_length(prompt_len)
        sess.set_pending(first_o)
        want = om.generate(first_o, 12, k, mask)
        got = sess.decode(12, k)
        assert np.array_equal(got["tokens"], want["tokens"]), f"k={k}: oracle min margin {want['min_margin']}"
        assert np.array_equal(got["accepts"], want["accepts"])


def test_config1_tiny_all_on_and_all_off_masks(kb):
    shape, om, sess = _pair(kb, "tiny", gain_spread=0.0)
    prompt = si.uniform_tokens(0, 0, 32, shape.vocab).numpy()
    _, first, _ = om.prefill(prompt)
    want = om.generate(first, 32, 4, np.zeros(8, np.uint8))
    sess.set_skipmask(np.zeros(8, np.uint8))
    got = sess.generate(prompt, 32, 4)
    assert np.array_equal(got["tokens"], want["tokens"]) and np.array_equal(got["accepts"], want["accepts"])
    assert got["stats"]["accepted"] == got["stats"]["drafted"]       # the draft model is the full model
    om2 = oracle.OracleModel(shape, om._keep, 160)
    _, first, _ = om2.prefill(prompt)
    want = om2.generate(first, 32, 4, np.ones(8, np.uint8))
    sess.set_skipmask(np.ones(8, np.uint8))
    got = sess.generate(prompt, 32, 4)
    assert np.array_equal(got["tokens"], want["tokens"]) and np.array_equal(got["accepts"], want["accepts"])


def test_generate_with_selection_uses_the_domain_mask(kb):
    base = si.SHAPES["ragged-bf16"]
    nd, per = 4, 5
    anchors = si.anchors(3, nd, per, base.d_model, 0.5, clustered=False)
    masks = np.stack([si.skip_mask(s, 2 * base.n_layers, 2) for s in range(nd)])
    shape, om, sess = _pair(kb, "ragged-bf16", anchors=anchors, masks=masks, per=per)
    prompt = si.uniform_tokens(4, 0, 27, shape.vocab).numpy()
    pooled, first, _ = om.prefill(prompt)
    dom, _, _ = oracle.knn_select(pooled, anchors.numpy(), nd, per)
    want = om.generate(first, 20, 4, masks[dom])
    got = sess.generate(prompt, 20, 4, use_selection=True)
    assert got["domain"] == dom
    assert np.array_equal(got["tokens"], want["tokens"]) and np.array_equal(got["accepts"], want["accepts"])


def test_last_token_pooling_mode(kb):
    shape, om, sess = _pair(kb, "tiny", pool_mode=1)
    prompt = si.uniform_tokens(0, 0, 19, shape.vocab).numpy()
    om.prefill(prompt[:18])
    want = om.forward(prompt[18:19], 18, want_hidden=True)["hidden"][0]
    _, pooled = sess.prefill(prompt, want_pooled=True)
    assert np.abs(pooled.cpu().numpy() - want).max() < 1e-4


# ---- protocol and error paths ---------------------------------------------------------------------

def test_protocol_errors_leave_the_session_usable(kb):
    shape, om, sess = _pair(kb, "tiny", max_seq=48, max_draft=4)
    E = kb.KnnssdError

    def status(fn, *a, **k):
        with pytest.raises(E) as e:
            fn(*a, **k)
        return e.value.status

    assert status(sess.draft, 2) == 4                              # before prefill
    assert status(sess.verify, [1, 2]) == 4
    assert status(sess.select_skipset) == 4                        # no anchors in this context
    assert status(sess.prefill, []) == 1
    assert status(sess.prefill, [5, shape.vocab]) == 1             # token id out of range
    assert status(sess.prefill, list(range(48))) == 3              # does not fit
    prompt = si.uniform_tokens(0, 0, 40, shape.vocab).numpy()
    first = sess.prefill(prompt)
    assert status(sess.draft, 2) == 4                              # no mask yet
    assert status(sess.set_skipmask, np.full(8, 2, np.uint8)) == 1
    sess.set_skipmask(si.skip_mask(0, 8, 3))
    assert status(sess.draft, 5) == 1                              # k > max_draft
    assert status(sess.draft, 0) == 1
    assert status(sess.verify, [shape.vocab]) == 1
    assert status(sess.generate, prompt, 16, 4) == 3               # 40 + 16 + 1 > 48
    assert status(sess.set_length, 41) == 1                        # rollback only
    assert sess.length == 40
    # after all those refusals the session still works and still agrees with the oracle
    _, first_o, _ = om.prefill(prompt)
    assert first == first_o
    d = sess.draft(4)
    r = sess.verify(d)
    o = om.forward(np.concatenate([[first], d]).astype(np.int32), 40)
    assert (r["n_accepted"], r["next_token"]) == oracle.accept(d, o["argmax"])


def test_init_rejects_unsupported_shapes(kb):
    shape = si.SHAPES["tiny"]
    w = _to_dev(si.make_model_weights(shape, 0))
    with pytest.raises(kb.KnnssdError) as e:
        kb.Session(n_layers=4, d_model=256, n_heads=8, n_kv_heads=8, head_dim=32, d_ff=688, vocab=1024, max_seq=64,
                   max_draft=4, rms_eps=1e-5, rope_theta=1e4, dtype="fp32", weights=w)
    assert e.value.status == 2
    with pytest.raises(kb.KnnssdError) as e:
        kb.Session(n_layers=4, d_model=256, n_heads=4, n_kv_heads=4, head_dim=64, d_ff=688, vocab=1024, max_seq=64,
                   max_draft=4, rms_eps=1e-5, rope_theta=1e4, dtype="fp32", weights=w,
                   anchors=torch.zeros((6, 256), device="cuda"), skip_masks=np.zeros((3, 8), np.uint8),
                   anchors_per_domain=2)
    assert e.value.status == 5                                      # zero anchors are degenerate


def test_rollback_then_replay_gives_the_same_tokens(kb):
    """Rows beyond the committed length are dead: rolling back and decoding again reproduces the tokens."""
    shape, om, sess = _pair(kb, "gqa-bf16")
    prompt = si.uniform_tokens(2, 0, 30, shape.vocab).numpy()
    first = sess.prefill(prompt)
    sess.set_skipmask(si.skip_mask(0, 4, 2))
    a = [sess.verify(sess.draft(4))["next_token"] for _ in range(3)]
    len_after = sess.length
    sess.set_length(30)
    sess.set_pending(first)
    b = [sess.verify(sess.draft(4))["next_token"] for _ in range(3)]
    assert a == b and sess.length == len_after


# ---- contexts beyond 2048 positions ------------------------------------------------------------------

@pytest.mark.parametrize("shape_name", ["stream64-bf16", "stream-bf16"])
def test_context_beyond_2048_positions_matches_oracle(kb, shape_name):
    """A 2100-token prompt (three chunks of the prompt pass; 33 attention segments, so the merge's second set of segment
    statistics is in use), then teacher-forced verification rows and a generated stretch against the live oracle."""
    P, max_seq = 2100, 2300
    base = si.SHAPES[shape_name]
    mask = si.skip_mask(0, 2 * base.n_layers, 2)
    damp = {int(j): 0.05 for j in np.nonzero(mask)[0]}
    shape, om, sess = _pair(kb, shape_name, max_seq=max_seq, damp=damp)
    prompt = si.uniform_tokens(3, 0, P, shape.vocab).numpy()
    pooled_o, first_o, _ = om.prefill(prompt)
    first_g, pooled_g = sess.prefill(prompt, want_pooled=True)
    assert first_g == first_o
    assert np.abs(pooled_g.cpu().numpy() - pooled_o).max() < TOL["bf16"]
    sess.set_skipmask(mask)
    n, pending = P, first_o
    forced = si.uniform_tokens(9, 1, 40, shape.vocab).numpy()
    fi = 0
    for k in (4, 8, 0, 2):
        rows = forced[fi:fi + k]
        fi += k
        o = om.forward(np.concatenate([[pending], rows]).astype(np.int32), n, want_hidden=True)
        g = sess.verify(rows, want_logits=True, want_hidden=True)
        assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < TOL["bf16"]
        assert np.abs(g["hidden"].cpu().numpy() - o["hidden"]).max() < TOL["bf16"]
        a, nxt = oracle.accept(rows, o["argmax"])
        assert (g["n_accepted"], g["next_token"]) == (a, nxt)
        n += a + 1
        om.length = n
        pending = nxt
    want = om.generate(pending, 20, 4, mask)
    got = sess.decode(20, 4)
    assert np.array_equal(got["tokens"], want["tokens"]), f"oracle min margin {want['min_margin']}"
    assert np.array_equal(got["accepts"], want["accepts"])
    assert sess.length == om.length > 2048 + 64


# ---- a row's numbers do not depend on how many rows its pass carries -------------------------------------------

@pytest.mark.parametrize("shape_name", ["stream-bf16", "stream64-bf16"])
def test_a_row_is_bit_identical_whatever_the_pass_carries(kb, shape_name):
    """The same token at the same position gives the same logits and hidden state, bit for bit, whether it is verified
    alone (1 row), with 1..3 more rows (the form that packs both terms of a row into one product), with 4..7 more (one
    product per term), in a pass of 9..12 rows (three packed products) or of 13..16: losslessness on the GPU rests on
    this."""
    shape, om, sess = _pair(kb, shape_name, max_seq=160, max_draft=15)
    prompt = si.uniform_tokens(5, 0, 70, shape.vocab).numpy()
    first = sess.prefill(prompt)
    rows = si.uniform_tokens(6, 1, 15, shape.vocab).numpy()
    ref = None
    for k in (0, 1, 3, 4, 7, 8, 11, 12, 15):
        sess.set_length(70)
        sess.set_pending(first)
        g = sess.verify(rows[:k], want_logits=True, want_hidden=True)
        if ref is None:
            ref = sess.verify  # placeholder to keep the first result below
            full = (g["logits"].clone(), g["hidden"].clone())
        else:
            assert torch.equal(g["logits"][0], full[0][0]) and torch.equal(g["hidden"][0], full[1][0]), f"k = {k}"
        if k == 15:
            wide = (g["logits"].clone(), g["hidden"].clone())
    # and the other rows of the widest pass against narrower passes that contain them
    for k in (1, 3, 4, 7, 8, 11, 12):
        sess.set_length(70)
        sess.set_pending(first)
        g = sess.verify(rows[:k], want_logits=True, want_hidden=True)
        assert torch.equal(g["logits"], wide[0][:k + 1]) and torch.equal(g["hidden"], wide[1][:k + 1]), f"k = {k}"
