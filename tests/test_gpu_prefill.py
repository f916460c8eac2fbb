"""The prompt pass on the tensor cores against the CPU oracle.

The contraction is checked on its own (all three epilogues, ragged row and unit counts, long inputs), then the whole
prompt pass through ``knnssd_prefill``: first token, pooled state and the tokens decoded from the K/V cache it leaves.
"""
import numpy as np
import pytest
import torch

import oracle
import synthetic_inputs as si

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def kb():
    if not torch.cuda.is_available():
        pytest.fail("the gpu tests need a CUDA device")
    from paper_2505_16162_b200 import build
    build.build()
    from paper_2505_16162_b200 import binding
    return binding


def _oracle_linear(W, x):
    """The oracle's linear map, 64 rows at a time (rows are independent)."""
    return np.concatenate([oracle.linear(W, x[i:i + 64]) for i in range(0, x.shape[0], 64)])


def _tol(n_in, want):
    """Two bf16 terms carry 16 mantissa bits of x (2e-5 of the largest output covers that, as for the decode kernel).
    The tensor core adds each 16-column product to its fp32 accumulator with truncation, one ulp of the running sum
    at most per step; a sum stays in tensor memory for a chunk of 512 columns only (64 steps of 2^-23 relative) and the
    chunks are added in registers with ordinary rounding (n_in / 512 steps of 2^-24).  An observed bound of this
    kernel's arithmetic, not one the method fixes; the whole-path tolerance on logits stays 2e-2."""
    return (2e-5 + 64 * 2.0 ** -23 + n_in / 512 * 2.0 ** -24) * max(1.0, float(np.abs(want).max()))


def _inputs(n_out, n_in, T, seed=3):
    W = si.normal_weight(seed, 77, n_out, n_in, 0.02, "bf16")
    x = si.normal_f32(seed + 1, 78, torch.arange(T * n_in), 1.0).view(T, n_in).contiguous()
    return W, x


# one tile; ragged rows and units (second weight box partly / wholly past the end, a column chunk cut short);
# several row tiles; the 13B-shaped widths; one row
GEMM_CASES = [(512, 256, 128), (1000, 320, 77), (136, 64, 5), (640, 1024, 300), (5120, 5120, 260), (264, 13824, 130),
              (15360, 5120, 1),
              # tile widths other than 128 columns (the launch picks the width with the fewest column-rounds on the
              # GPU's SMs): 192, 320 and 256 on a 148-SM part
              (5120, 256, 520), (5120, 256, 900), (4608, 256, 1024),
              # more tiles than SMs (a CTA walks several tiles); a ragged last tile
              (5120, 2176, 900), (4936, 512, 1000),
              # 320-column tiles on three rotating accumulators (picked where they save a round and the input is long
              # enough to pay for their one-tile CTAs): staggered chunks with short last ones (69 k-blocks), a ragged
              # last tile (136 of 320 columns, a weight box partly past the end)
              (4936, 4416, 900)]


@pytest.mark.parametrize("n_out,n_in,T", GEMM_CASES)
def test_gemm_store_matches_oracle(kb, n_out, n_in, T):
    W, x = _inputs(n_out, n_in, T)
    want = _oracle_linear(W, x.numpy())
    got = kb.knnssd_gemm_split(W.cuda(), x.cuda(), 0).cpu().numpy()
    assert np.abs(got - want).max() < _tol(n_in, want)


@pytest.mark.parametrize("n_out,n_in,T", [(1000, 320, 77), (5120, 5120, 260), (4936, 4416, 900)])
def test_gemm_add_matches_oracle(kb, n_out, n_in, T):
    W, x = _inputs(n_out, n_in, T)
    y0 = si.normal_f32(9, 79, torch.arange(T * n_out), 1.0).view(T, n_out).contiguous()
    want = y0.numpy().astype(np.float64) + _oracle_linear(W, x.numpy())
    got = kb.knnssd_gemm_split(W.cuda(), x.cuda(), 1, y=y0.clone().cuda()).cpu().numpy()
    assert np.abs(got - want).max() < _tol(n_in, want)


@pytest.mark.parametrize("n_out,n_in,T", [(1000, 320, 77), (13824, 5120, 140), (200, 256, 128), (2304, 128, 1024)])
def test_gemm_swiglu_matches_oracle(kb, n_out, n_in, T):
    Wg, x = _inputs(n_out, n_in, T)
    Wu = si.normal_weight(11, 80, n_out, n_in, 0.02, "bf16")
    g = _oracle_linear(Wg, x.numpy()).astype(np.float64)
    u = _oracle_linear(Wu, x.numpy()).astype(np.float64)
    want = g / (1.0 + np.exp(-g)) * u
    got = kb.knnssd_gemm_split(Wg.cuda(), x.cuda(), 2, W1=Wu.cuda()).cpu().numpy()
    # the result is handed on as two bf16 terms: 16 mantissa bits
    assert np.abs(got - want).max() < 1.5 * _tol(n_in, want)


def test_gemm_rows_do_not_depend_on_the_batch(kb):
    """A row's result is the same whichever rows share its tile."""
    W, x = _inputs(520, 384, 200)
    full = kb.knnssd_gemm_split(W.cuda(), x.cuda(), 0)
    part = kb.knnssd_gemm_split(W.cuda(), x[130:131].contiguous().cuda(), 0)
    assert torch.equal(part[0], full[130])


def test_gemm_rejects_bad_arguments(kb):
    W = torch.zeros((16, 96), dtype=torch.bfloat16, device="cuda")
    x = torch.zeros((2, 96), device="cuda")
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_gemm_split(W, x, 0)                     # n_in not a multiple of 64
    assert e.value.status == 2
    W = torch.zeros((12, 128), dtype=torch.bfloat16, device="cuda")
    x = torch.zeros((2, 128), device="cuda")
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_gemm_split(W, x, 0)                     # n_out not a multiple of 8
    assert e.value.status == 2
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_gemm_split(torch.zeros((16, 128), dtype=torch.bfloat16, device="cuda"), x, 2)   # SwiGLU without W1
    assert e.value.status == 1


# ---- the whole prompt pass ---------------------------------------------------------------------------

TOL = 2e-2          # bf16 weights and K/V: the tolerance of the decode-path tests


def _to_dev(w):
    return {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}


def _pair(kb, shape_name, max_seq, max_draft=8, pool_mode=0, damp=None):
    shape = si.SHAPES[shape_name]
    w = si.make_model_weights(shape, 0, gain_spread=0.1, damp=damp)
    om = oracle.OracleModel(shape, w, max_seq)
    sess = kb.Session.from_shape(shape, _to_dev(w), max_seq, max_draft=max_draft, pool_mode=pool_mode)
    return shape, om, sess


# prompt lengths: just past one pass's rows, one ragged tile, two tiles and a tail, three tiles exactly
@pytest.mark.parametrize("prompt_len", [17, 100, 300, 384])
@pytest.mark.parametrize("shape_name", ["stream-bf16", "stream64-bf16"])
def test_prompt_pass_matches_oracle(kb, shape_name, prompt_len):
    """First token and pooled state of the prompt pass, then - reading the K/V cache it left - the logits and final
    hidden states of a verification pass over forced rows, and the tokens generated from there."""
    shape, om, sess = _pair(kb, shape_name, prompt_len + 80)
    prompt = si.uniform_tokens(5, 0, prompt_len, shape.vocab).numpy()
    pooled_o, first_o, _ = om.prefill(prompt)
    first_g, pooled_g = sess.prefill(prompt, want_pooled=True)
    assert first_g == first_o
    assert np.abs(pooled_g.cpu().numpy() - pooled_o).max() < TOL
    rows = si.uniform_tokens(6, 1, 7, shape.vocab).numpy()
    o = om.forward(np.concatenate([[first_o], rows]).astype(np.int32), prompt_len, want_hidden=True)
    sess.set_skipmask(np.zeros(2 * shape.n_layers, dtype=np.uint8))
    g = sess.verify(rows, want_logits=True, want_hidden=True)
    assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < TOL
    assert np.abs(g["hidden"].cpu().numpy() - o["hidden"]).max() < TOL
    a, nxt = oracle.accept(rows, o["argmax"])
    assert (g["n_accepted"], g["next_token"]) == (a, nxt)


@pytest.mark.parametrize("shape_name", ["stream-bf16", "stream64-bf16"])
def test_generate_after_a_long_prompt_matches_oracle_exactly(kb, shape_name):
    base = si.SHAPES[shape_name]
    mask = si.skip_mask(0, 2 * base.n_layers, 2)
    damp = {int(j): 0.05 for j in np.nonzero(mask)[0]}
    shape, om, sess = _pair(kb, shape_name, 300, damp=damp)
    prompt = si.uniform_tokens(2, 0, 200, shape.vocab).numpy()
    _, first, _ = om.prefill(prompt)
    want = om.generate(first, 40, 4, mask)
    sess.set_skipmask(mask)
    got = sess.generate(prompt, 40, 4)
    assert np.array_equal(got["tokens"], want["tokens"]), f"oracle min margin {want['min_margin']}"
    assert np.array_equal(got["accepts"], want["accepts"])


@pytest.mark.parametrize("n_prompt", [1025, 1100])
def test_prompt_longer_than_one_chunk(kb, n_prompt):
    """More than 1024 prompt rows: the second chunk (a single row, or 76) reads the first chunk's K/V from the cache."""
    shape, om, sess = _pair(kb, "stream64-bf16", 1200)
    prompt = si.uniform_tokens(3, 0, n_prompt, shape.vocab).numpy()
    pooled_o, first_o, _ = om.prefill(prompt)
    first_g, pooled_g = sess.prefill(prompt, want_pooled=True)
    assert first_g == first_o
    assert np.abs(pooled_g.cpu().numpy() - pooled_o).max() < TOL
    o = om.forward(np.array([first_o], dtype=np.int32), n_prompt)
    sess.set_skipmask(np.zeros(2 * shape.n_layers, dtype=np.uint8))
    g = sess.verify(np.zeros(0, dtype=np.int32), want_logits=True)
    assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < TOL
    assert g["next_token"] == int(o["argmax"][0])


def test_last_token_pooling_after_the_prompt_pass(kb):
    shape, om, sess = _pair(kb, "stream-bf16", 200, pool_mode=1)
    prompt = si.uniform_tokens(4, 0, 90, shape.vocab).numpy()
    _, first_o, _ = om.prefill(prompt)
    first_g, pooled_g = sess.prefill(prompt, want_pooled=True)
    assert first_g == first_o
    h = om.forward(prompt[-1:], 89, want_hidden=True, want_logits=False)["hidden"][0]   # K/V of rows 0..88 are in place
    assert np.abs(pooled_g.cpu().numpy() - h).max() < TOL


def test_sixteen_row_pass_matches_oracle(kb):
    """The widest pass the decode kernel takes (two blocks of 8 rows): 15 forced rows after the pending token."""
    shape, om, sess = _pair(kb, "stream-bf16", 120, max_draft=15)
    prompt = si.uniform_tokens(0, 0, 37, shape.vocab).numpy()
    _, first_o, _ = om.prefill(prompt)
    assert sess.prefill(prompt) == first_o
    sess.set_skipmask(np.zeros(2 * shape.n_layers, dtype=np.uint8))
    for n_rows in (15, 9):
        rows = si.uniform_tokens(7, n_rows, n_rows, shape.vocab).numpy()
        n = sess.length
        om.length = n                                       # rows the last verification rejected are dead
        o = om.forward(np.concatenate([[first_o], rows]).astype(np.int32), n, want_hidden=True)
        g = sess.verify(rows, want_logits=True, want_hidden=True)
        assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < TOL
        assert np.abs(g["hidden"].cpu().numpy() - o["hidden"]).max() < TOL
        a, nxt = oracle.accept(rows, o["argmax"])
        assert (g["n_accepted"], g["next_token"]) == (a, nxt)
        first_o = nxt                                       # the pending token of the next round


# ---- the mask-search objective (Sec. 4.1, Eq. (3)) -------------------------------------------------------

def test_mask_objective_counts_match_oracle(kb):
    """f(z) is a time, so the oracle cannot give its value; what it fixes is what was timed: for every candidate
    mask and sample the accepted / drafted totals of the decode loop must be the oracle's, and the value must be the
    per-token time of exactly those rounds."""
    shape, om, sess = _pair(kb, "stream-bf16", 200)
    L2 = 2 * shape.n_layers
    masks = np.stack([np.zeros(L2, dtype=np.uint8), si.skip_mask(0, L2, 2), si.skip_mask(1, L2, 3)])
    prompts = [si.uniform_tokens(20 + i, 0, n, shape.vocab).numpy() for i, n in enumerate((21, 60))]
    max_new, k = 20, 4
    ms, acc, drf = sess.mask_objective(masks, prompts, max_new, k)
    want_acc, want_drf = np.zeros(3, dtype=np.int64), np.zeros(3, dtype=np.int64)
    for p in prompts:
        for m in range(3):
            _, first, _ = om.prefill(p)
            r = om.generate(first, max_new, k, masks[m])
            want_acc[m] += r["accepted"]
            want_drf[m] += r["drafted"]
    assert np.array_equal(acc, want_acc) and np.array_equal(drf, want_drf)
    assert acc[0] == drf[0]                                   # nothing skipped: the draft model is the full model
    assert (ms > 0).all()
    # the session is left usable, with the last mask active
    assert len(sess.decode(5, 2)["tokens"]) == 5


@pytest.mark.parametrize("shape_name", ["stream-bf16", "stream64-bf16"])
def test_every_row_count_of_the_common_kernel_with_grouped_heads(kb, shape_name):
    """Verification passes of 1..8 rows on GQA shapes (3 and 4 query heads per K/V head): an attention task then
    carries up to 8 of the (head, row) pairs of a K/V head and a group spans several tasks."""
    shape, om, sess = _pair(kb, shape_name, 200)
    prompt = si.uniform_tokens(1, 0, 70, shape.vocab).numpy()       # the last segment starts inside the prompt
    _, first_o, _ = om.prefill(prompt)
    assert sess.prefill(prompt) == first_o
    sess.set_skipmask(np.zeros(2 * shape.n_layers, dtype=np.uint8))
    pending = first_o
    for n_rows in (7, 6, 5, 0, 3):
        rows = si.uniform_tokens(30 + n_rows, 2, n_rows, shape.vocab).numpy() if n_rows else np.zeros(0, dtype=np.int32)
        n = sess.length
        om.length = n
        o = om.forward(np.concatenate([[pending], rows]).astype(np.int32), n, want_hidden=True)
        g = sess.verify(rows, want_logits=True, want_hidden=True)
        assert np.abs(g["logits"].cpu().numpy() - o["logits"]).max() < TOL
        assert np.abs(g["hidden"].cpu().numpy() - o["hidden"]).max() < TOL
        a, nxt = oracle.accept(rows, o["argmax"])
        assert (g["n_accepted"], g["next_token"]) == (a, nxt)
        pending = nxt


# ---- weight-streaming linear map for up to 16 rows on the tensor cores (stand-alone) ------------------------

@pytest.mark.parametrize("n_out,n_in,M", [(5120, 5120, 1), (5120, 5120, 16), (1003, 320, 9), (15360, 5120, 5), (130, 13824, 16),
                                          (40000, 384, 7), (96, 64, 3)])
def test_linear_tc_matches_oracle(kb, n_out, n_in, M):
    W, x = _inputs(n_out, n_in, M)
    want = _oracle_linear(W, x.numpy())
    got, ms = kb.knnssd_linear_tc(W.cuda(), x.cuda())
    assert np.abs(got.cpu().numpy() - want).max() < _tol(n_in, want)
    assert ms > 0


def test_linear_tc_rows_do_not_depend_on_the_batch_and_limits(kb):
    W, x = _inputs(1003, 384, 16)
    full, _ = kb.knnssd_linear_tc(W.cuda(), x.cuda())
    for M in (1, 5, 9):
        part, _ = kb.knnssd_linear_tc(W.cuda(), x[:M].contiguous().cuda())
        assert torch.equal(part, full[:M])
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_linear_tc(W.cuda(), torch.zeros((17, 384), device="cuda"))
    assert e.value.status == 3
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_linear_tc(torch.zeros((8, 96), dtype=torch.bfloat16, device="cuda"), torch.zeros((1, 96), device="cuda"))
    assert e.value.status == 2
