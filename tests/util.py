"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI binding, run the
oracle on the same seeded inputs (fed the GPU's fp32 logits so that routing decisions are taken
on identical numbers), and compare tensor by tensor."""
import numpy as np
import torch

from oracle import btx_oracle as o
from paper_2403_07816_b200 import binding as B
from paper_2403_07816_b200 import synth

TOL = {torch.float32: 1e-5, torch.bfloat16: 1e-2}     # max|err| / max|ref| per output tensor


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    denom = np.max(np.abs(ref))
    if denom == 0.0:
        return float(np.max(np.abs(got)))
    return float(np.max(np.abs(got - ref)) / denom)


def gpu_forward(inp, k, routing=B.ROUTE_TOPK, alpha=0.01, bias=None, save=True, stopgrad_u=False, skip_wgrad=False,
                noise=None, tau=0.0, capacity_factor=0.0):
    x = inp["x"]
    T, d = x.shape
    E, F, _ = inp["w1"].shape
    desc = B.make_desc(T, d, F, E, k, x.dtype, routing, alpha, stopgrad_u, save, skip_wgrad, tau, capacity_factor)
    ws, saved = B.alloc_buffers(desc, x.device)
    ws.fill_(0x7F)           # poison: results must not depend on scratch contents
    saved.fill_(0x7F)
    r = B.Routing.empty(desc, x.device)
    y = torch.empty_like(x)
    B.btx_moe_forward(desc, x, inp["w_router"], bias, inp["w1"], inp["w3"], inp["w2"], y, r, saved if save else None, ws,
                      router_noise=noise)
    assert B.btx_device_status(ws) == B.BTX_OK
    return dict(desc=desc, y=y, routing=r, saved=saved, ws=ws, noise=noise, tau=tau)


def gpu_backward(inp, fwd, lb_scale=1.0, bias=None, accumulate=False, init=None):
    x = inp["x"]
    desc = fwd["desc"]
    E, F, d = inp["w1"].shape
    dev = x.device
    mk = (lambda *s: torch.full(s, init, dtype=torch.float32, device=dev)) if init is not None else \
         (lambda *s: torch.empty(s, dtype=torch.float32, device=dev))
    out = dict(dx=torch.empty_like(x), dw_router=mk(E, d), dbias=mk(E))
    if desc.skip_wgrad:
        out.update(dw1=None, dw3=None, dw2=None)
    else:
        out.update(dw1=mk(E, F, d), dw3=mk(E, F, d), dw2=mk(E, d, F))
    fwd["ws"].fill_(0x7F)
    B.btx_moe_backward(desc, x, inp["w_router"], bias, inp["w1"], inp["w3"], inp["w2"], inp["dy"], lb_scale,
                       fwd["saved"], out["dx"], out["dw_router"], out["dbias"], out["dw1"], out["dw3"], out["dw2"],
                       int(accumulate), fwd["ws"], router_noise=fwd.get("noise"))
    assert B.btx_device_status(fwd["ws"]) == B.BTX_OK
    return out


def np64(t):
    return synth.to_f64_numpy(t)


def check_forward(inp, fwd, k, routing, alpha, bias, tol, noise=None, tau=1.0, capacity_factor=0.0):
    """Parity protocol: logits by tolerance; routing and permutation bit-exact given the GPU's
    fp32 logits; gates, probabilities, loss and y by tolerance."""
    r = fwd["routing"]
    cpu = {n: np64(t) for n, t in inp.items()}
    b64 = None if bias is None else np64(bias)
    z_ref = o.router_logits(cpu["x"], cpu["w_router"], b64)
    z_gpu = r.logits.cpu().numpy()
    assert rel_err(z_gpu, z_ref) <= tol, "logits"
    n64 = None if noise is None else np64(noise)
    ref = o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], k, routing, alpha,
                        router_bias=b64, logits=z_gpu, noise=n64, tau=tau, capacity_factor=capacity_factor)
    for name, got in [("topk_idx", r.topk_idx), ("counts", r.counts), ("offsets", r.offsets), ("perm", r.perm),
                      ("inv_perm", r.inv_perm)]:
        assert np.array_equal(got.cpu().numpy(), ref[name]), name
    assert rel_err(r.gates.cpu().numpy(), ref["gates"]) <= tol, "gates"
    assert rel_err(r.probs.cpu().numpy(), ref["probs"]) <= tol, "probs"
    assert rel_err(r.u.cpu().numpy(), ref["u"]) <= tol, "u"
    assert rel_err(r.p.cpu().numpy(), ref["p"]) <= tol, "p"
    assert abs(float(r.lb_loss.item()) - ref["lb_loss"]) <= tol * max(abs(ref["lb_loss"]), 1e-30), "lb_loss"
    e = rel_err(np64(fwd["y"]), ref["y"])
    assert e <= tol, f"y rel err {e}"
    return cpu, b64, z_gpu, ref


def check_backward(cpu, b64, z_gpu, got, k, routing, alpha, lb_scale, stopgrad_u, tol, base=None, noise=None, tau=1.0,
                   capacity_factor=0.0):
    n64 = None if noise is None else np64(noise)
    ref = o.moe_backward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], cpu["dy"], k, routing, alpha,
                         lb_scale, stopgrad_u, router_bias=b64, logits=z_gpu, noise=n64, tau=tau,
                         capacity_factor=capacity_factor)
    errs = {}
    for name in ("dx", "dw_router", "dbias", "dw1", "dw3", "dw2"):
        if got[name] is None:
            continue
        want = ref[name] if base is None or name == "dx" else ref[name] + base
        errs[name] = rel_err(np64(got[name]), want)
    bad = {n: e for n, e in errs.items() if e > tol}
    assert not bad, f"backward rel errs over {tol}: {bad} (all: {errs})"
    return errs
