"""The allocation-free top-k entry point (scratch inside the library image) must give what the
regular entry point gives with a caller workspace.  Collected last on purpose: if it fails, a run
that stops at the first failure has already run everything else.

Who needs it: a caller that receives only input and output buffers and cannot get more device
memory when the call is made (a plug-in with a frozen memory pool, a decode step that must not
call cudaMalloc).  The test uses few rows so that rows are split into segments, which is the case
that needs scratch at all."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2608_27514_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _outputs(n, k):
    return (torch.empty(n, dtype=torch.float32, device=DEV), torch.empty((n, k), dtype=torch.int32, device=DEV),
            torch.empty((n, k), dtype=torch.float32, device=DEV), torch.empty(n, dtype=torch.float32, device=DEV))


def _regular(x, k):
    n, V = x.shape
    out = _outputs(n, k)
    need = B.tsd_confidence_topk_workspace_bytes(n, V, k)
    assert need > 0, "this shape is meant to need scratch"
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    B.tsd_confidence_topk(x, k, *out, workspace=ws)
    torch.cuda.synchronize()
    return out


def _static(x, k):
    out = _outputs(x.shape[0], k)
    B.tsd_confidence_topk_static(x, k, *out)
    torch.cuda.synchronize()
    return out


def _check_against_oracle(x, k, got):
    host = x.float().cpu().numpy() if x.dtype == torch.bfloat16 else x.cpu().numpy()
    r_conf, r_idx, r_prob, r_lse = oracle.confidence_topk(host, k)
    assert np.array_equal(got[1].cpu().numpy(), r_idx)                       # indices: bit-exact
    assert np.abs(got[0].cpu().numpy() - r_conf).max() <= 1e-5
    assert np.abs(got[2].cpu().numpy() - r_prob).max() <= 1e-5
    assert np.abs(got[3].cpu().numpy() - r_lse).max() <= 1e-4


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    g = torch.Generator(device=DEV).manual_seed(77)
    k = 3
    # different inputs back to back: each call finds the previous call's leftovers in the shared
    # array and must not be affected by them.  The shapes differ in segments per row and in k, so
    # that the partial-result slots of one call overlap the ticket words of another, and both
    # element types take part.
    xa = (torch.randn((100, 126464), generator=g, device=DEV) * 3).bfloat16()
    xb = (torch.randn((40, 50000), generator=g, device=DEV) * 3).bfloat16()
    xc = torch.randn((7, 90000), generator=g, device=DEV) * 3                  # fp32
    xd = (torch.randn((3, 300000), generator=g, device=DEV) * 3).bfloat16()
    assert 0 < B.tsd_confidence_topk_workspace_bytes(100, 126464, k) <= B.tsd_confidence_topk_static_capacity()
    for x, kk in ((xa, k), (xb, k), (xc, 8), (xa, k), (xd, 1), (xc, 2)):
        ref = _regular(x, kk)
        got = _static(x, kk)
        assert torch.equal(got[1], ref[1])                         # indices: bit-exact
        for a, b in ((got[0], ref[0]), (got[2], ref[2])):          # probabilities: the suite's 1e-5
            assert (a - b).abs().max().item() <= 1e-5
        assert (got[3] - ref[3]).abs().max().item() <= 1e-4
        _check_against_oracle(x, kk, got)                          # and the definition itself


def test_static_scratch_rejects_what_does_not_fit():
    # long rows force every one of many rows into several segments: 4.4 MB of partial results,
    # more than the 1 MiB the library carries, so the call must be refused before any launch
    n, V, k = 20000, 300000, 8
    need = B.tsd_confidence_topk_workspace_bytes(n, V, k)
    assert need > B.tsd_confidence_topk_static_capacity()
    x = torch.zeros((1, 16), dtype=torch.bfloat16, device=DEV)     # never read: the call is refused first
    out = _outputs(1, k)
    rc = B.lib().tsd_confidence_topk_static(
        ctypes.c_void_p(x.data_ptr()), B.TSD_BF16, n, V, V, k, ctypes.c_void_p(out[0].data_ptr()),
        ctypes.c_void_p(out[1].data_ptr()), ctypes.c_void_p(out[2].data_ptr()), None, None, None)
    assert rc == B.TSD_ERR_WORKSPACE
