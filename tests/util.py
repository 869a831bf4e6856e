"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI binding, run the
oracle on the same seeded inputs (fed the GPU's fp32 logits so that routing decisions are taken
on identical numbers), and compare tensor by tensor."""
import numpy as np
import torch

from oracle import btx_oracle as o
from paper_2403_07816_b200 import binding as B
from paper_2403_07816_b200 import synth

TOL = {torch.float32: 1e-5, torch.bfloat16: 1e-2}     # max|err| / max|ref| per output tensor

# Guard bands.  Every buffer the library writes (workspace, saved state, outputs) is carved out of a
# larger allocation with GUARD bytes of a fixed pattern on both sides; after each call the bands must
# still hold the pattern.  An index that runs past a buffer (a padded row count, a split count, a tile
# of a ragged shape) lands in a band and fails the test instead of silently corrupting a neighbour.
GUARD = 4096
GUARD_BYTE = 0xA5


class Guarded:
    def __init__(self, shape, dtype, device, fill=None):
        shape = tuple(int(v) for v in (shape if isinstance(shape, (tuple, list)) else (shape,)))
        n = 1
        for v in shape:
            n *= v
        self.nbytes = n * torch.empty((), dtype=dtype).element_size()
        inner = (max(self.nbytes, 16) + 255) // 256 * 256          # keeps the rear band 256-byte aligned
        self.raw = torch.full((GUARD + inner + GUARD,), GUARD_BYTE, dtype=torch.uint8, device=device)
        self.t = self.raw[GUARD:GUARD + self.nbytes].view(dtype).view(shape)
        self.inner = inner
        # what the library does not write stays visible: NaN patterns in floating-point buffers, a large
        # positive number in integer ones (an unwritten index would not pass for the -1 "dropped" mark)
        self.raw[GUARD:GUARD + self.nbytes].fill_(0xFF if dtype.is_floating_point else 0x7F)
        if fill is not None:
            self.t.fill_(fill)

    def intact(self):
        front = self.raw[:GUARD]
        back = self.raw[GUARD + self.nbytes:]
        return bool((front == GUARD_BYTE).all()) and bool((back == GUARD_BYTE).all())


def check_guards(bufs, where):
    torch.cuda.synchronize()
    for name, g in bufs.items():
        assert g.intact(), f"{where}: bytes outside `{name}` were overwritten"


def guarded_routing(desc, device, bufs):
    k = desc.E if desc.routing == B.ROUTE_SOFT else desc.k
    T, E, R = desc.T, desc.E, desc.T * k
    f, i = torch.float32, torch.int32
    spec = [("logits", (T, E), f), ("topk_idx", (T, k), i), ("gates", (T, k), f), ("probs", (T, E), f),
            ("counts", (E,), i), ("offsets", (E + 1,), i), ("perm", (R,), i), ("inv_perm", (R,), i), ("u", (E,), f),
            ("p", (E,), f), ("lb_loss", (1,), f)]
    ts = []
    for name, shape, dt in spec:
        bufs["routing." + name] = Guarded(shape, dt, device)
        ts.append(bufs["routing." + name].t)
    return B.Routing(*ts)


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
    ws_bytes, saved_bytes = B.btx_moe_sizes(desc)
    bufs = {}
    # poison (0x7F): results must not depend on scratch contents
    bufs["workspace"] = Guarded(ws_bytes, torch.uint8, x.device, fill=0x7F)
    bufs["saved"] = Guarded(max(saved_bytes, 16), torch.uint8, x.device, fill=0x7F)
    bufs["y"] = Guarded(x.shape, x.dtype, x.device)
    ws, saved, y = bufs["workspace"].t, bufs["saved"].t, bufs["y"].t
    r = guarded_routing(desc, x.device, bufs)
    B.btx_moe_forward(desc, x, inp["w_router"], bias, inp["w1"], inp["w3"], inp["w2"], y, r, saved if save else None, ws,
                      router_noise=noise)
    assert B.btx_device_status(ws) == B.BTX_OK
    check_guards(bufs, "forward")
    return dict(desc=desc, y=y, routing=r, saved=saved, ws=ws, noise=noise, tau=tau, bufs=bufs)


def gpu_backward(inp, fwd, lb_scale=1.0, bias=None, accumulate=False, init=None):
    x = inp["x"]
    desc = fwd["desc"]
    E, F, d = inp["w1"].shape
    dev = x.device
    bufs = dict(fwd["bufs"])                      # the forward's buffers are watched during the backward as well

    def mk(name, *shape):
        bufs[name] = Guarded(shape, torch.float32, dev, fill=init)
        return bufs[name].t
    bufs["dx"] = Guarded(x.shape, x.dtype, dev)
    out = dict(dx=bufs["dx"].t, dw_router=mk("dw_router", E, d), dbias=mk("dbias", E))
    bufs["dlogits"] = Guarded((x.shape[0], E), torch.float32, dev)
    out["dlogits"] = bufs["dlogits"].t
    if desc.skip_wgrad:
        out.update(dw1=None, dw3=None, dw2=None)
    else:
        out.update(dw1=mk("dw1", E, F, d), dw3=mk("dw3", E, F, d), dw2=mk("dw2", E, d, F))
    fwd["ws"].fill_(0x7F)
    B.btx_moe_backward(desc, x, inp["w_router"], bias, inp["w1"], inp["w3"], inp["w2"], inp["dy"], lb_scale,
                       fwd["saved"], out["dx"], out["dw_router"], out["dbias"], out["dw1"], out["dw3"], out["dw2"],
                       int(accumulate), fwd["ws"], router_noise=fwd.get("noise"), dlogits=out["dlogits"])
    assert B.btx_device_status(fwd["ws"]) == B.BTX_OK
    check_guards(bufs, "backward")
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
                        router_bias=b64, logits=z_gpu, noise=n64, tau=tau, capacity_factor=capacity_factor,
                        select_fp32=True)
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
                         capacity_factor=capacity_factor, select_fp32=True)
    errs = {}
    for name in ("dx", "dw_router", "dlogits", "dw1", "dw3", "dw2"):
        if got.get(name) is None:
            continue
        want = ref[name] if base is None or name in ("dx", "dlogits") else ref[name] + base
        errs[name] = rel_err(np64(got[name]), want)
    bad = {n: e for n, e in errs.items() if e > tol}
    assert not bad, f"backward rel errs over {tol}: {bad} (all: {errs})"
    # dbias = sum_t dz_t is a sum of mixed-sign terms that can cancel to far below their size (with two
    # experts its two entries are +s and -s), so max|ref| is not a meaningful scale for its rounding error.
    # Its bar is the same tolerance taken relative to the size of what was summed, max_e sum_t |dz_t,e|,
    # from the oracle's own dz (the design notes list this as a reading of the tolerance).
    want = ref["dbias"] if base is None else ref["dbias"] + base
    err_abs = float(np.max(np.abs(np64(got["dbias"]) - want)))
    scale = float(np.max(np.sum(np.abs(ref["dlogits"]), axis=0)))
    errs["dbias"] = rel_err(np64(got["dbias"]), want)             # reported: the plain max-norm figure
    errs["dbias_vs_summed_size"] = err_abs / scale if scale > 0 else err_abs
    assert errs["dbias_vs_summed_size"] <= tol, f"dbias {errs}"
    return errs
