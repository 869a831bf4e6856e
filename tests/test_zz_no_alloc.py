"""btx_lb_loss_noalloc: the load-balancing loss for callers that cannot allocate device memory
(plug-ins living inside another framework's memory pool, loops that must avoid cudaMalloc's
device-wide synchronisation).  Its scratch is a static array inside the library, shared by all
calls and never cleaned between them, so the check runs it on several shapes in a row (large then
small, with the expert count and k changed, so that the later calls find the earlier ones' leftovers
inside the regions they use) and holds every run to the CPU oracle's fp64 loss and gradient; the
ordinary workspace-taking entry point runs the same kernels and must agree bit for bit.
Collected last on purpose: a failure here cannot hide another test."""
import numpy as np
import pytest
import torch

from oracle import btx_oracle as o
from paper_2403_07816_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-5                       # the FP32 bar of the other tests: max|err| / max|ref| per output


def _outputs(T, E, with_grad=True):
    out = [torch.full((1,), 9.0, device=DEV), torch.full((E,), 9.0, device=DEV), torch.full((E,), 9.0, device=DEV)]
    out.append(torch.full((T, E), 9.0, device=DEV) if with_grad else None)
    return out


def _rel(got, want):
    got, want = np.asarray(got, dtype=np.float64), np.asarray(want, dtype=np.float64)
    return float(np.max(np.abs(got - want)) / max(np.max(np.abs(want)), 1e-30))


def _check_against_oracle(out, z, k, routing, alpha):
    E = z.shape[1]
    kk = E if routing == B.ROUTE_SOFT else k
    loss, u, p = o.lb_loss_from_logits(z, kk, routing, alpha)
    assert abs(float(out[0].item()) - loss) <= TOL * abs(loss)
    assert _rel(out[1].cpu().numpy(), u) <= TOL and _rel(out[2].cpu().numpy(), p) <= TOL
    if out[3] is not None:
        assert _rel(out[3].cpu().numpy(), o.lb_loss_grad(z, kk, routing, alpha)) <= TOL


def test_noalloc_matches_the_oracle_on_calls_in_a_row_that_share_the_scratch():
    g = torch.Generator(device="cpu").manual_seed(21)
    # (T, E, k, routing, bias): large first, then smaller shapes whose scratch regions lie inside what it dirtied
    cases = [(24000, 8, 2, B.ROUTE_TOPK, False), (777, 4, 2, B.ROUTE_TOPK, True), (2048, 8, 1, B.ROUTE_SWITCH, False),
             (5, 3, 3, B.ROUTE_SOFT, False), (777, 4, 2, B.ROUTE_TOPK, False)]
    for T, E, k, routing, with_bias in cases:
        logits = (torch.randn(T, E, generator=g) * 1.5).to(DEV)
        bias = (torch.randn(E, generator=g) * 0.5).to(DEV) if with_bias else None
        desc = B.make_desc(T, 0, 0, E, k, torch.float32, routing, 0.01)
        assert B.btx_lb_loss_workspace_size(desc) <= (4 << 20)
        z = ((logits + bias) if with_bias else logits).cpu().numpy()          # the fp32 sum the kernel forms
        got = _outputs(T, E)
        B.btx_lb_loss_noalloc(desc, logits, *got, router_bias=bias)
        torch.cuda.synchronize()
        _check_against_oracle(got, z, k, routing, 0.01)
        # same kernels on a caller-owned workspace: identical bits
        ws = torch.empty(B.btx_lb_loss_workspace_size(desc), dtype=torch.uint8, device=DEV)
        want = _outputs(T, E)
        B.btx_lb_loss(desc, logits, *want, ws, router_bias=bias)
        torch.cuda.synchronize()
        for a, b in zip(got, want):
            assert torch.equal(a, b)
        # loss only (no gradient requested), again on the dirty scratch
        lean = _outputs(T, E, with_grad=False)
        B.btx_lb_loss_noalloc(desc, logits, *lean, router_bias=bias)
        torch.cuda.synchronize()
        _check_against_oracle(lean, z, k, routing, 0.01)
        for a, b in zip(lean[:3], got[:3]):
            assert torch.equal(a, b)


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    T, E = 1 << 20, 8
    desc = B.make_desc(T, 0, 0, E, 2, torch.float32, B.ROUTE_TOPK, 0.01)
    assert B.btx_lb_loss_workspace_size(desc) > (4 << 20)
    logits = torch.zeros(8, E, device=DEV)              # never read: the call must fail before any launch
    out = torch.zeros(8, device=DEV)
    with pytest.raises(B.BtxError) as ei:
        B.btx_lb_loss_noalloc(desc, logits, out, out, out, None)
    assert ei.value.status == 3
    # the largest request it takes and the smallest it refuses are told apart by the size query alone
    for T in (40000, 43000, 50000):
        d4 = B.make_desc(T, 0, 0, 4, 2, torch.float32, B.ROUTE_TOPK, 0.01)
        fits = B.btx_lb_loss_workspace_size(d4) <= (4 << 20)
        lg = torch.zeros(T, 4, device=DEV)
        outs = _outputs(T, 4, with_grad=False)
        if fits:
            B.btx_lb_loss_noalloc(d4, lg, *outs)
            torch.cuda.synchronize()
            assert abs(float(outs[0].item()) - 0.01) < 1e-7      # all logits tie: L_LB = alpha exactly
        else:
            with pytest.raises(B.BtxError) as ei:
                B.btx_lb_loss_noalloc(d4, lg, *outs)
            assert ei.value.status == 3
