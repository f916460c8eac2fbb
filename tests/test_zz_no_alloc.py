"""The allocation-free cosine search against the ordinary one and against the CPU oracle (collected last on purpose).

Some callers cannot call cudaMalloc: a serving loop that lives inside a memory pool sized at start-up, a process
under a fixed GPU memory reservation, a latency path that cannot afford cudaFree's implicit synchronisation.
``knnssd_cosine_top1_static`` serves them by keeping its scratch in a fixed array inside the library.  That array is
shared by every call and keeps the previous call's contents, so the check is made on two calls in a row whose
inputs differ in size and in outcome: whatever the first call left behind must not leak into the second.
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


def _same(kb, query, anchors):
    want = kb.knnssd_cosine_top1(query, anchors)
    got = kb.knnssd_cosine_top1_static(query, anchors)
    assert got[0] == want[0]
    assert abs(got[1] - want[1]) < 1e-5          # the tolerance the cosine parity tests use; same kernels, so equal
    # ... and both against the oracle's Eq. (4) on the same inputs (one domain holding all the anchors)
    dom, anc, cs = oracle.knn_select(query.cpu().numpy(), anchors.cpu().numpy(), 1, anchors.shape[0])
    assert got[0] == anc and abs(got[1] - cs) < 1e-5
    return got


def test_static_scratch_variant_matches_on_two_calls_in_a_row(kb):
    a = si.anchors(0, 5, 10, 5120, 0.2).cuda()
    big = si.anchors(1, 40, 25, 640, 0.5, clustered=False).cuda()            # 1000 anchors: fills far more scratch
    q_big = si.normal_f32(3, 11, torch.arange(640), 1.0).cuda()
    # call 1: many anchors; call 2: few anchors of another dimension - stale cosines beyond n must not win
    _same(kb, q_big, big)
    best, cos = _same(kb, (2.5 * a[17]).contiguous(), a)
    assert best == 17 and abs(cos - 1.0) < 1e-5
    # a degenerate query raises the flag word in the shared array; the next call must start from a cleared flag
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_cosine_top1_static(torch.zeros(5120, device="cuda"), a)
    assert e.value.status == 5
    _same(kb, a[3].contiguous(), a)
    _same(kb, q_big, big)


def test_static_scratch_variant_refuses_more_anchors_than_it_holds(kb):
    n = kb.STATIC_MAX_ANCHORS + 1
    anchors = torch.ones((n, 8), device="cuda")
    q = torch.ones(8, device="cuda")
    with pytest.raises(kb.KnnssdError) as e:
        kb.knnssd_cosine_top1_static(q, anchors)
    assert e.value.status == 3
    # at the limit it still works and agrees with the allocating call and the oracle (all cosines equal: lowest index wins)
    assert _same(kb, q, anchors[:-1].contiguous())[0] == 0
    with pytest.raises(ValueError):                   # the binding refuses a query shorter than the anchors' rows
        kb.knnssd_cosine_top1_static(q[:4].contiguous(), anchors[:-1].contiguous())
