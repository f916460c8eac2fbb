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
    """Two bf16 terms carry 16 mantissa bits of x (2e-5 of the largest output covers that, as for the decode kernel);
    the tensor core adds each 16-column product to its fp32 accumulator with truncation, one ulp of the running sum
    at most per step: n_in / 16 steps of 2^-23 relative."""
    return (2e-5 + n_in / 16 * 2.0 ** -23) * max(1.0, float(np.abs(want).max()))


def _inputs(n_out, n_in, T, seed=3):
    W = si.normal_weight(seed, 77, n_out, n_in, 0.02, "bf16")
    x = si.normal_f32(seed + 1, 78, torch.arange(T * n_in), 1.0).view(T, n_in).contiguous()
    return W, x


# one tile; ragged rows and units (second weight box partly / wholly past the end, a column chunk cut short);
# several row tiles; the 13B-shaped widths; one row
GEMM_CASES = [(512, 256, 128), (1000, 320, 77), (136, 64, 5), (640, 1024, 300), (5120, 5120, 260), (264, 13824, 130),
              (15360, 5120, 1)]


@pytest.mark.parametrize("n_out,n_in,T", GEMM_CASES)
def test_gemm_store_matches_oracle(kb, n_out, n_in, T):
    W, x = _inputs(n_out, n_in, T)
    want = _oracle_linear(W, x.numpy())
    got = kb.knnssd_gemm_split(W.cuda(), x.cuda(), 0).cpu().numpy()
    assert np.abs(got - want).max() < _tol(n_in, want)


@pytest.mark.parametrize("n_out,n_in,T", [(1000, 320, 77), (5120, 5120, 260)])
def test_gemm_add_matches_oracle(kb, n_out, n_in, T):
    W, x = _inputs(n_out, n_in, T)
    y0 = si.normal_f32(9, 79, torch.arange(T * n_out), 1.0).view(T, n_out).contiguous()
    want = y0.numpy().astype(np.float64) + _oracle_linear(W, x.numpy())
    got = kb.knnssd_gemm_split(W.cuda(), x.cuda(), 1, y=y0.clone().cuda()).cpu().numpy()
    assert np.abs(got - want).max() < _tol(n_in, want)


@pytest.mark.parametrize("n_out,n_in,T", [(1000, 320, 77), (13824, 5120, 140), (200, 256, 128)])
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
