"""btx_lb_loss_noalloc: the load-balancing loss for callers that cannot allocate device memory
(plug-ins living inside another framework's memory pool, loops that must avoid cudaMalloc's
device-wide synchronisation).  Its scratch is a static array inside the library, shared by all
calls, so the check runs it twice in a row and compares both runs with the ordinary
workspace-taking entry point.  Collected last on purpose: a failure here cannot hide another test."""
import numpy as np
import pytest
import torch

from paper_2403_07816_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _run(fn_noalloc, desc, logits):
    T, E = logits.shape
    out = [torch.full((1,), 9.0, device=DEV), torch.full((E,), 9.0, device=DEV), torch.full((E,), 9.0, device=DEV),
           torch.full((T, E), 9.0, device=DEV)]
    if fn_noalloc:
        B.btx_lb_loss_noalloc(desc, logits, *out)
    else:
        ws = torch.empty(B.btx_lb_loss_workspace_size(desc), dtype=torch.uint8, device=DEV)
        B.btx_lb_loss(desc, logits, *out, ws)
    torch.cuda.synchronize()
    return [t.cpu().numpy().astype(np.float64) for t in out]


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    g = torch.Generator(device="cpu").manual_seed(21)
    cases = [(777, 4, 2, B.ROUTE_TOPK), (2048, 8, 1, B.ROUTE_SWITCH)]     # second call reuses a dirty scratch
    for T, E, k, routing in cases:
        logits = (torch.randn(T, E, generator=g) * 1.5).to(DEV)
        desc = B.make_desc(T, 0, 0, E, k, torch.float32, routing, 0.01)
        want = _run(False, desc, logits)
        got = _run(True, desc, logits)
        for a, b in zip(got, want):
            denom = max(np.max(np.abs(b)), 1e-30)
            assert np.max(np.abs(a - b)) / denom <= 1e-5


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    T, E = 1 << 20, 8
    desc = B.make_desc(T, 0, 0, E, 2, torch.float32, B.ROUTE_TOPK, 0.01)
    assert B.btx_lb_loss_workspace_size(desc) > (4 << 20)
    logits = torch.zeros(8, E, device=DEV)              # never read: the call must fail before any launch
    o = torch.zeros(8, device=DEV)
    with pytest.raises(B.BtxError) as ei:
        B.btx_lb_loss_noalloc(desc, logits, o, o, o, None)
    assert ei.value.status == 3
