"""Device-side failure paths of the C ABI, in their bounded form: nothing here faults, traps or hangs a GPU.

* KNNSSD_ERR_TIMEOUT: every wait in the kernels has a poll limit.  The test hook launches the persistent pass kernel
  with a grid barrier that cannot complete and a limit of a few thousand polls; every CTA gives up, the kernel returns
  and the call reports status 7.  Afterwards the same context must work again and agree with the oracle.
* non-finite logits: a model whose final norm gains are NaN yields logit rows without any finite value; the arg-max
  then has nothing to choose, must still return an id inside the vocabulary (no out-of-range gather later) and the
  call reports KNNSSD_ERR_DEGENERATE.
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


def _to_dev(w):
    return {k: ([t.cuda() for t in v] if isinstance(v, list) else v.cuda()) for k, v in w.items()}


def test_a_wait_that_runs_out_reports_timeout_and_the_context_recovers(kb):
    shape = si.SHAPES["stream-bf16"]
    mask = si.skip_mask(0, 2 * shape.n_layers, 3)
    damp = {int(j): 0.05 for j in np.nonzero(mask)[0]}
    w = si.make_model_weights(shape, 0, damp=damp, gain_spread=0.1)
    om = oracle.OracleModel(shape, w, 160)
    prompt = si.uniform_tokens(0, 0, 37, shape.vocab).numpy()
    _, first, _ = om.prefill(prompt)
    want = om.generate(first, 24, 4, mask)
    sess = kb.Session.from_shape(shape, _to_dev(w), 160, max_draft=4)
    sess.set_skipmask(mask)
    got = sess.generate(prompt, 24, 4)
    assert np.array_equal(got["tokens"], want["tokens"])
    for spin_limit in (2000, 6000):
        with pytest.raises(kb.KnnssdError) as e:
            sess.debug_barrier_timeout(spin_limit)
        assert e.value.status == 7
        # the failed pass invalidated the session: the next decode call is refused until a new prefill
        with pytest.raises(kb.KnnssdError) as e:
            sess.draft(2)
        assert e.value.status == 4
        got = sess.generate(prompt, 24, 4)
        assert np.array_equal(got["tokens"], want["tokens"]) and np.array_equal(got["accepts"], want["accepts"])
    with pytest.raises(kb.KnnssdError) as e:
        sess.debug_barrier_timeout(0)
    assert e.value.status == 1


def test_timeout_hook_is_refused_where_the_persistent_kernel_does_not_run(kb):
    shape = si.SHAPES["tiny"]
    sess = kb.Session.from_shape(shape, _to_dev(si.make_model_weights(shape, 0)), 64, max_draft=4)
    with pytest.raises(kb.KnnssdError) as e:
        sess.debug_barrier_timeout(2000)
    assert e.value.status == 2


@pytest.mark.parametrize("shape_name", ["tiny", "stream-bf16"])
def test_logits_without_a_finite_value_are_reported_not_followed(kb, shape_name):
    shape = si.SHAPES[shape_name]
    w = si.make_model_weights(shape, 0)
    good = _to_dev(w)
    bad = dict(good)
    bad["final_norm"] = torch.full_like(good["final_norm"], float("nan"))
    sess = kb.Session.from_shape(shape, bad, 96, max_draft=4)
    prompt = si.uniform_tokens(0, 0, 20, shape.vocab).numpy()
    with pytest.raises(kb.KnnssdError) as e:
        sess.prefill(prompt)
    assert e.value.status == 5
    with pytest.raises(kb.KnnssdError) as e:
        sess.set_skipmask(np.zeros(2 * shape.n_layers, np.uint8))
        sess.generate(prompt, 8, 2)
    assert e.value.status == 5
    sess.close()
    # the same weights with a finite norm still decode and agree with the oracle: the error left nothing behind
    om = oracle.OracleModel(shape, w, 96)
    _, first, _ = om.prefill(prompt)
    mask = si.skip_mask(0, 2 * shape.n_layers, 2)
    want = om.generate(first, 8, 2, mask)
    ok = kb.Session.from_shape(shape, good, 96, max_draft=4)
    ok.set_skipmask(mask)
    got = ok.generate(prompt, 8, 2)
    assert np.array_equal(got["tokens"], want["tokens"])
