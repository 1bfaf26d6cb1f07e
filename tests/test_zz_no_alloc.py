"""GPU test of grace_beam_topk_static, the top-k entry point that brings its own scratch memory.

It exists for callers that cannot allocate device memory where they need the selection (they are
handed input and output buffers and nothing else), so the test gives it exactly that: inputs and
outputs, no workspace.  Its results must equal those of grace_beam_topk (indices exactly, scores
bit for bit) on two calls in a row with different inputs -- the second call sees whatever the
first left in the shared scratch.  Collected last (file name) so that a failure here cannot hide
the other tests; it also passes when run alone in a fresh process.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _outputs(B, K):
    return (torch.empty((B, K), device=DEV), torch.empty((B, K), dtype=torch.int32, device=DEV),
            torch.empty((B, K), dtype=torch.int32, device=DEV), torch.empty((B, K), dtype=torch.int32, device=DEV))


def _both(api, cand, K, V):
    B, N = cand.shape
    ws = torch.empty(api.grace_beam_topk_workspace_bytes(B, N, K), dtype=torch.uint8, device=DEV)
    ref = _outputs(B, K)
    api.grace_beam_topk(cand, K, V, *ref, ws)
    got = _outputs(B, K)
    for t in got:
        t.fill_(-7)
    api.grace_beam_topk_static(cand, K, V, *got)
    torch.cuda.synchronize()
    return ref, got


def _assert_same(ref, got):
    assert torch.equal(ref[0].view(torch.int32), got[0].view(torch.int32))      # scores, bit for bit
    for a, b in zip(ref[1:], got[1:]):
        assert torch.equal(a, b)


def test_static_scratch_topk_matches_workspace_topk_twice_in_a_row():
    from paper_2608_00938_b200 import api
    g = torch.Generator(device=DEV)
    g.manual_seed(260800938 + 4000)
    # first call: sampled path (large N), dense scores, the maximum number of requests
    B, V, K = api.grace_beam_topk_static_max_requests(), 1024, 2048
    cand1 = torch.randn(B, 300 * V, device=DEV, generator=g) * 3.0 - 8.0
    _assert_same(*_both(api, cand1, K, V))
    # second call right after: other shape, mostly -inf (underfull beams) and exact ties, fewer requests
    cand2 = torch.randn(5, 320 * V, device=DEV, generator=g)
    cand2[torch.rand(cand2.shape, device=DEV, generator=g) < 0.997] = float("-inf")
    cand2[0, :5000] = 0.5
    _assert_same(*_both(api, cand2, 1500, V))
    # and a small-N call that takes the exact single-CTA path
    cand3 = torch.randn(3, 64 * 64, device=DEV, generator=g)
    _assert_same(*_both(api, cand3, 16, 64))


def test_static_scratch_topk_rejects_more_requests_than_it_holds():
    from paper_2608_00938_b200 import api
    B = api.grace_beam_topk_static_max_requests() + 1
    cand = torch.zeros(B, 4096, device=DEV)
    with pytest.raises(api.GraceError) as err:
        api.grace_beam_topk_static(cand, 8, 64, *_outputs(B, 8))
    assert "workspace too small" in str(err.value)
