"""Pins of the CPU oracle against things other than itself (no GPU).

Each test ties one part of the oracle to a library routine, a closed form, an
invariant or brute force, chosen so that a dropped term, a wrong sign or index,
or a transposed operand fails at least one of them.
"""
import itertools
import math

import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as si


def _model(shape_name, seed=0, max_seq=96, gain_spread=0.1, damp=None):
    shape = si.SHAPES[shape_name]
    w = si.make_model_weights(shape, seed, gain_spread=gain_spread, damp=damp)
    return shape, w, oracle.OracleModel(shape, w, max_seq)


def _as_f64(t):
    return t.to(torch.float32).to(torch.float64)


def _library_decoder(shape, w):
    """The standard transformer-library LLaMA decoder (the one the paper's stack runs,
    App. C.1) holding the same weights, evaluated in fp64."""
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg = LlamaConfig(hidden_size=shape.d_model, intermediate_size=shape.d_ff,
                      num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
                      num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim,
                      vocab_size=shape.vocab, rms_norm_eps=shape.rms_eps, rope_theta=shape.rope_theta,
                      attention_bias=False, mlp_bias=False, tie_word_embeddings=False,
                      max_position_embeddings=4096)
    cfg._attn_implementation = "eager"
    m = LlamaForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": _as_f64(w["tok_embed"]),
          "model.norm.weight": _as_f64(w["final_norm"]),
          "lm_head.weight": _as_f64(w["lm_head"])}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj",
             "wo": "self_attn.o_proj", "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj",
             "w_down": "mlp.down_proj", "attn_norm": "input_layernorm", "mlp_norm": "post_attention_layernorm"}
    for l in range(shape.n_layers):
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}.weight"] = _as_f64(w[k][l])
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and all("rotary" in k or "inv_freq" in k for k in missing), (missing, unexpected)
    return m


@pytest.mark.parametrize("shape_name", ["tiny", "gqa-fp32"])
def test_decoder_matches_library_llama(shape_name):
    shape, w, om = _model(shape_name)
    ref = _library_decoder(shape, w)
    toks = si.uniform_tokens(3, 0, 40, shape.vocab).numpy()
    with torch.no_grad():
        want = ref(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    # rows enter in uneven chunks so that later rows attend to cached K/V of earlier calls
    got = np.concatenate([om.forward(toks[a:b], a)["logits"] for a, b in [(0, 16), (16, 17), (17, 40)]])
    assert np.abs(got - want).max() < 2e-5
    # the final-norm hidden state is what the head sees: W_lm . hidden == logits
    hid = om.forward(toks[:8], 0, want_hidden=True)["hidden"]
    lm = _as_f64(w["lm_head"]).numpy()
    assert np.abs(hid.astype(np.float64) @ lm.T - want[:8]).max() < 2e-5


def test_bf16_model_matches_library_llama_within_cache_rounding():
    shape, w, om = _model("gqa-bf16")
    ref = _library_decoder(shape, w)
    toks = si.uniform_tokens(4, 0, 24, shape.vocab).numpy()
    with torch.no_grad():
        want = ref(torch.tensor(toks[None].astype(np.int64))).logits[0].numpy()
    got = om.forward(toks, 0)["logits"]
    err = np.abs(got - want).max()
    assert 0 < err < 5e-3          # K/V rounded to bf16 in the cache: close, not identical


def test_single_position_attention_returns_v_rounded_to_bf16():
    """softmax over one position is 1, so the attention output is the cached V row:
    with bf16 storage the result must equal the fp64 library result computed with V
    rounded to bf16, and differ from the unrounded one."""
    shape = si.SHAPES["gqa-bf16"].with_layers(1)
    w = si.make_model_weights(shape, 5, gain_spread=0.1)
    om = oracle.OracleModel(shape, w, 8)
    tok = np.array([7], dtype=np.int32)
    got = om.forward(tok, 0)["logits"][0].astype(np.float64)
    d, hd, H, Hkv = shape.d_model, shape.head_dim, shape.n_heads, shape.n_kv_heads
    x = _as_f64(w["tok_embed"])[7]

    def norm(v, g):
        return v / torch.sqrt((v * v).mean() + shape.rms_eps) * _as_f64(g)

    def full(round_v):
        v = _as_f64(w["wv"][0]) @ norm(x, w["attn_norm"][0])
        if round_v:
            v = v.to(torch.float32).to(torch.bfloat16).to(torch.float64)
        o = v.view(Hkv, 1, hd).expand(Hkv, H // Hkv, hd).reshape(H * hd)
        y = x + _as_f64(w["wo"][0]) @ o
        h = norm(y, w["mlp_norm"][0])
        g, u = _as_f64(w["w_gate"][0]) @ h, _as_f64(w["w_up"][0]) @ h
        y = y + _as_f64(w["w_down"][0]) @ (torch.nn.functional.silu(g) * u)
        return (_as_f64(w["lm_head"]) @ norm(y, w["final_norm"])).numpy()

    assert np.abs(got - full(True)).max() < 2e-6
    assert np.abs(got - full(False)).max() > 1e-5


@pytest.mark.parametrize("shape_name", ["tiny", "gqa-bf16"])
def test_rows_at_once_equal_rows_one_by_one(shape_name):
    """Verification over k+1 rows in one pass is the same function as k+1 single-row steps."""
    shape, w, om = _model(shape_name)
    toks = si.uniform_tokens(1, 0, 21, shape.vocab).numpy()
    a = om.forward(toks[:12], 0)["logits"]
    b = om.forward(toks[12:], 12)["logits"]
    om2 = oracle.OracleModel(shape, w, 96)
    one = np.concatenate([om2.forward(toks[i:i + 1], i)["logits"] for i in range(21)])
    assert np.array_equal(np.concatenate([a, b]), one)


def test_all_skipped_mask_is_head_on_normed_embedding():
    shape, w, om = _model("tiny")
    toks = np.array([5, 900, 17], dtype=np.int32)
    mask = np.ones(2 * shape.n_layers, dtype=np.uint8)
    got = om.forward(toks, 0, skip_mask=mask)["logits"].astype(np.float64)
    x = _as_f64(w["tok_embed"])[toks.astype(np.int64)]
    h = x / torch.sqrt((x * x).mean(dim=1, keepdim=True) + shape.rms_eps) * _as_f64(w["final_norm"])
    want = (h @ _as_f64(w["lm_head"]).T).numpy()
    assert np.abs(got - want).max() < 2e-6


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_skipping_a_sublayer_equals_zeroing_its_output_projection(seed):
    """z^(j) = 1 removes sublayer j's residual branch: the full model with that
    sublayer's output projection set to zero gives the same logits, bit for bit."""
    shape = si.SHAPES["tiny"]
    mask = si.skip_mask(seed, 2 * shape.n_layers, 3)
    w = si.make_model_weights(shape, 0, gain_spread=0.1)
    toks = si.uniform_tokens(2, 0, 9, shape.vocab).numpy()
    got = oracle.OracleModel(shape, w, 32).forward(toks, 0, skip_mask=mask)["logits"]
    wz = si.make_model_weights(shape, 0, gain_spread=0.1)
    for j in np.nonzero(mask)[0]:
        (wz["wo"] if j % 2 == 0 else wz["w_down"])[j // 2].zero_()
    want = oracle.OracleModel(shape, wz, 32).forward(toks, 0)["logits"]
    assert np.array_equal(got, want)
    assert not np.array_equal(got, oracle.OracleModel(shape, w, 32).forward(toks, 0)["logits"])


def test_all_retained_mask_is_the_full_model():
    shape, w, om = _model("tiny")
    toks = si.uniform_tokens(2, 0, 6, shape.vocab).numpy()
    a = om.forward(toks, 0, skip_mask=np.zeros(2 * shape.n_layers, dtype=np.uint8))["logits"]
    b = oracle.OracleModel(shape, w, 32).forward(toks, 0)["logits"]
    assert np.array_equal(a, b)


# ---- selection -------------------------------------------------------------------------------

def test_pool_is_the_mean():
    rng = np.random.default_rng(0)
    h = rng.standard_normal((37, 19)).astype(np.float32)
    assert np.allclose(oracle.pool_mean(h), h.astype(np.float64).mean(axis=0), rtol=0, atol=1e-7)
    row = rng.standard_normal(19).astype(np.float32)
    assert np.array_equal(oracle.pool_mean(np.tile(row, (8, 1))), row)


def test_knn_matches_brute_force_cosine():
    rng = np.random.default_rng(1)
    for trial in range(50):
        nd, per, d = int(rng.integers(1, 6)), int(rng.integers(1, 9)), int(rng.integers(2, 40))
        a = rng.standard_normal((nd * per, d)).astype(np.float32) * rng.uniform(0.1, 10, (nd * per, 1)).astype(np.float32)
        v = rng.standard_normal(d).astype(np.float32)
        a64, v64 = a.astype(np.float64), v.astype(np.float64)
        cos = (a64 @ v64) / (np.linalg.norm(a64, axis=1) * np.linalg.norm(v64))
        dom, anc, cs = oracle.knn_select(v, a, nd, per)
        flat = dom * per + anc
        assert cos[flat] >= cos.max() - 1e-6
        assert abs(cs - cos.max()) < 1e-6
        assert 0 <= dom < nd and 0 <= anc < per


def test_knn_closed_forms():
    a = si.anchors(0, 3, 8, 256, 0.1).numpy()
    for flat in (0, 5, 23):
        dom, anc, cs = oracle.knn_select(3.7 * a[flat], a, 3, 8)
        assert (dom, anc) == (flat // 8, flat % 8) and abs(cs - 1.0) < 1e-6
    rng = np.random.default_rng(2)
    v = rng.standard_normal(256).astype(np.float32)
    base = oracle.knn_select(v, a, 3, 8)
    for c in (1e-3, 0.5, 40.0):
        r = oracle.knn_select(c * v, a, 3, 8)
        assert r[:2] == base[:2] and abs(r[2] - base[2]) < 1e-6
    opposite = oracle.knn_select(-a[4], a, 3, 8)
    assert opposite[:2] != (0, 4)
    # ties go to the lowest flat index; degenerate inputs are reported, not guessed
    dup = np.concatenate([a[:3], a[:3]])
    assert oracle.knn_select(a[1], dup, 2, 3)[:2] == (0, 1)
    assert oracle.knn_select(np.zeros(256, np.float32), a, 3, 8) is None
    bad = a.copy()
    bad[7] = 0
    assert oracle.knn_select(v, bad, 3, 8) is None


def test_knn_separated_clusters_are_always_classified_correctly():
    """Clearly separated clusters give 100 % domain accuracy (Sec. 5.3)."""
    nd, per, d = 5, 10, 512
    a = si.anchors(7, nd, per, d, 0.2).numpy()
    cen = si.domain_centroids(7, nd, d).numpy()
    rng = np.random.default_rng(3)
    for i in range(200):
        dom = i % nd
        q = (cen[dom] + 0.3 * rng.standard_normal(d)).astype(np.float32)
        assert oracle.knn_select(q, a, nd, per)[0] == dom


# ---- acceptance and the speculative loop --------------------------------------------------------

def test_accept_rule_brute_force():
    for k in range(0, 4):
        for draft in itertools.product(range(2), repeat=k):
            for target in itertools.product(range(2), repeat=k + 1):
                a = 0
                for j in range(k + 1):      # largest j whose first j draft tokens all agree
                    if all(target[i] == draft[i] for i in range(j)):
                        a = j
                assert oracle.accept(draft, target) == (a, target[a])


def _run(shape_name, mask, k, max_new, prompt_len=12, seed=0, damp=None, max_seq=128):
    shape, w, om = _model(shape_name, seed=seed, max_seq=max_seq, damp=damp)
    prompt = si.uniform_tokens(seed, 0, prompt_len, shape.vocab).numpy()
    _, first, _ = om.prefill(prompt)
    spec = om.generate(first, max_new, k, mask)
    om2 = oracle.OracleModel(shape, w, max_seq)
    _, first2, _ = om2.prefill(prompt)
    plain, _ = om2.greedy_full(first2, max_new)
    return shape, spec, plain, first, first2


@pytest.mark.parametrize("k", [1, 2, 4, 8])
@pytest.mark.parametrize("mask_kind", ["seeded", "all_on", "all_off", "attn_only", "damped"])
def test_speculative_output_is_plain_greedy_output(k, mask_kind):
    """Losslessness (Sec. 1, Sec. 3.1, Sec. 7): whatever the mask and k, the tokens are those
    of plain greedy decoding with the full model."""
    L = si.SHAPES["tiny"].n_layers
    damp = None
    if mask_kind == "seeded":
        mask = si.skip_mask(0, 2 * L, 3)
    elif mask_kind == "all_on":
        mask = np.zeros(2 * L, np.uint8)
    elif mask_kind == "all_off":
        mask = np.ones(2 * L, np.uint8)
    elif mask_kind == "attn_only":
        mask = np.array([0, 1] * L, np.uint8)
    else:
        mask = si.skip_mask(0, 2 * L, 3)
        damp = {int(j): 0.02 for j in np.nonzero(mask)[0]}
    max_new = 23
    shape, spec, plain, f1, f2 = _run("tiny", mask, k, max_new, damp=damp)
    assert f1 == f2
    assert np.array_equal(spec["tokens"], plain)
    acc = spec["accepts"]
    assert all(0 <= a <= k for a in acc)                       # 1 <= tokens per pass <= k+1
    assert int(sum(a + 1 for a in acc)) + 1 == max_new
    assert spec["accepted"] == int(acc.sum())
    if mask_kind == "all_on":                                  # the draft model is the full model
        assert spec["rounds"] == math.ceil((max_new - 1) / (k + 1))
        assert spec["accepted"] == spec["drafted"]
    if mask_kind == "damped":                                  # skipped sublayers matter little: drafts often agree
        assert spec["accepted"] >= 0.3 * spec["drafted"]
    # accept counts recomputed by brute force from the plain greedy sequence
    pos = 1
    for r, a in enumerate(acc):
        drafts = [t for t in spec["drafts"][r] if t >= 0]
        agree = 0
        while agree < len(drafts) and pos + agree < max_new and drafts[agree] == plain[pos + agree]:
            agree += 1
        assert a == agree
        pos += a + 1


def test_last_round_never_overshoots():
    for max_new in (1, 2, 3, 6, 7):
        _, spec, plain, _, _ = _run("tiny", np.zeros(8, np.uint8), 4, max_new)
        assert len(spec["tokens"]) == max_new and np.array_equal(spec["tokens"], plain)


def test_bf16_gqa_loop_is_lossless():
    mask = si.skip_mask(1, 4, 2)
    _, spec, plain, _, _ = _run("gqa-bf16", mask, 3, 14, prompt_len=20)
    assert np.array_equal(spec["tokens"], plain)


# ---- the greedy choice and the cache's rounding points ----------------------------------------------

def test_greedy_choice_is_the_arg_max_of_the_logits():
    """Drafting equation of Sec. 4.2: the token is arg max of the logits.  The oracle's choice and its margin are
    compared with numpy's on the logits it returns (full model and a masked draft model)."""
    shape, w, om = _model("tiny")
    toks = si.uniform_tokens(6, 0, 24, shape.vocab).numpy()
    for mask in (None, si.skip_mask(0, 2 * shape.n_layers, 3)):
        o = oracle.OracleModel(shape, w, 32).forward(toks, 0, skip_mask=mask)
        lg = o["logits"]
        assert np.array_equal(o["argmax"], np.argmax(lg, axis=1))
        assert len(set(o["argmax"].tolist())) > 4              # not a constant
        top2 = np.sort(lg, axis=1)[:, -2:]
        assert np.array_equal(o["margin"], top2[:, 1] - top2[:, 0])
        assert (o["margin"] > 0).all()
    # only the last head_rows rows get a choice
    o = oracle.OracleModel(shape, w, 32).forward(toks[:5], 0, head_rows=2)
    assert (o["argmax"][:3] == -1).all() and np.array_equal(o["argmax"][3:], np.argmax(o["logits"][3:], axis=1))


def test_equal_logits_go_to_the_lowest_token_id():
    """Head rows v and v + V/2 are made identical, so every logit value occurs twice: the lower id must win and the
    margin is zero."""
    shape = si.SHAPES["tiny"]
    w = si.make_model_weights(shape, 0, gain_spread=0.1)
    half = shape.vocab // 2
    w["lm_head"][half:] = w["lm_head"][:half]
    om = oracle.OracleModel(shape, w, 32)
    toks = si.uniform_tokens(8, 0, 12, shape.vocab).numpy()
    o = om.forward(toks, 0)
    lg = o["logits"]
    assert np.array_equal(lg[:, :half], lg[:, half:])
    assert (o["argmax"] < half).all()
    assert np.array_equal(o["argmax"], np.argmax(lg[:, :half], axis=1))
    assert (o["margin"] == 0).all()
    # ... and the generation loop follows the same rule
    _, first, _ = om.prefill(toks)
    assert first < half
    out = om.generate(first, 9, 2, si.skip_mask(0, 2 * shape.n_layers, 3))
    assert (out["tokens"] < half).all() and out["min_margin"] == 0


def test_two_position_attention_sees_k_and_v_rounded_to_bf16():
    """One layer, two positions: the second row's softmax weighs both cached positions, so the result depends on the
    cached K.  It must equal the fp64 recomputation with the rotated K and V both rounded to bf16 on entering the
    cache, and differ from the one in which only V is rounded."""
    shape = si.SHAPES["gqa-bf16"].with_layers(1)
    w = si.make_model_weights(shape, 5, gain_spread=0.1)
    w["wq"][0] = w["wq"][0] * 4                                # exact in bf16; spreads the two scores apart
    w["wk"][0] = w["wk"][0] * 4
    om = oracle.OracleModel(shape, w, 8)
    toks = np.array([7, 11], dtype=np.int32)
    got = om.forward(toks, 0)["logits"][1].astype(np.float64)
    d, hd, H, Hkv = shape.d_model, shape.head_dim, shape.n_heads, shape.n_kv_heads

    def norm(v, g):
        return v / torch.sqrt((v * v).mean(dim=-1, keepdim=True) + shape.rms_eps) * _as_f64(g)

    def turn(v, pos):          # v [heads][hd]; dimension i pairs with i + hd/2
        i = torch.arange(hd // 2, dtype=torch.float64)
        ang = pos * shape.rope_theta ** (-2.0 * i / hd)
        a, b = v[:, :hd // 2], v[:, hd // 2:]
        return torch.cat([a * torch.cos(ang) - b * torch.sin(ang), b * torch.cos(ang) + a * torch.sin(ang)], dim=1)

    def through_cache(t, on):
        return t.to(torch.float32).to(torch.bfloat16).to(torch.float64) if on else t

    def full(round_k, round_v=True):
        x = _as_f64(w["tok_embed"])[toks.astype(np.int64)]
        h = norm(x, w["attn_norm"][0])
        q = turn((_as_f64(w["wq"][0]) @ h[1]).view(H, hd), 1)
        ks = torch.stack([through_cache(turn((_as_f64(w["wk"][0]) @ h[p]).view(Hkv, hd), p), round_k) for p in (0, 1)])
        vs = torch.stack([through_cache((_as_f64(w["wv"][0]) @ h[p]).view(Hkv, hd), round_v) for p in (0, 1)])
        g = H // Hkv
        o = torch.zeros(H, hd, dtype=torch.float64)
        for j in range(H):
            s = (ks[:, j // g] @ q[j]) / math.sqrt(hd)
            p = torch.softmax(s, dim=0)
            o[j] = p @ vs[:, j // g]
        y = x[1] + _as_f64(w["wo"][0]) @ o.reshape(H * hd)
        hm = norm(y, w["mlp_norm"][0])
        y = y + _as_f64(w["w_down"][0]) @ (torch.nn.functional.silu(_as_f64(w["w_gate"][0]) @ hm)
                                          * (_as_f64(w["w_up"][0]) @ hm))
        return (_as_f64(w["lm_head"]) @ norm(y, w["final_norm"])).numpy()

    assert np.abs(got - full(True)).max() < 2e-6
    assert np.abs(got - full(False)).max() > 1e-5
    assert np.abs(got - full(True, round_v=False)).max() > 1e-5
