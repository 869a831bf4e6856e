"""ctypes binding of libbtx.so: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (torch supplies device memory and streams); every step of the
layer runs inside the library.  There is no CPU fallback: if the library is missing or the
tensors are not on a CUDA device the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

BTX_OK = 0
BTX_ERR_INVALID_ARG, BTX_ERR_UNSUPPORTED, BTX_ERR_WORKSPACE, BTX_ERR_ARCH, BTX_ERR_CUDA, BTX_ERR_TIMEOUT = 1, 2, 3, 4, 5, 6
BTX_F32, BTX_BF16 = 0, 1
ROUTE_TOPK, ROUTE_SWITCH, ROUTE_SOFT, ROUTE_SAMPLE1 = 0, 1, 2, 3
PARAM_AVERAGE, PARAM_FFN = 0, 1
FFN_STACK, FFN_SPLIT, FFN_BLEND = 0, 1, 2

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbtx.so")
_lib = None


class BtxError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        msg = lib().btx_status_string(self.status).decode()
        super().__init__(f"{where}: {msg} (status {self.status})")


class MoeDesc(C.Structure):
    _fields_ = [("T", C.c_int32), ("d_model", C.c_int32), ("d_ff", C.c_int32), ("E", C.c_int32), ("k", C.c_int32),
                ("dtype", C.c_int32), ("routing", C.c_int32), ("lb_alpha", C.c_float),
                ("lb_stopgrad_u", C.c_int32), ("save_for_backward", C.c_int32), ("skip_wgrad", C.c_int32),
                ("gumbel_tau", C.c_float), ("capacity_factor", C.c_float)]


class RoutingOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("logits", "topk_idx", "gates", "probs", "counts", "offsets", "perm",
                                           "inv_perm", "u", "p", "lb_loss")]


class MergeItem(C.Structure):
    _fields_ = [("kind", C.c_int32), ("layer", C.c_int32), ("numel", C.c_uint64),
                ("src", C.POINTER(C.c_void_p)), ("dst", C.c_void_p)]


EXPORTS = ["btx_moe_sizes", "btx_moe_forward", "btx_moe_backward", "btx_moe_step_host",
           "btx_lb_loss_workspace_size", "btx_lb_loss", "btx_lb_loss_noalloc", "btx_merge_workspace_size", "btx_merge", "btx_merge_ffn_workspace_size", "btx_merge_ffn",
           "btx_device_status", "btx_selftest_wait_expiry", "btx_set_stage_events", "btx_status_string", "btx_version"]


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2403_07816_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32, sz = C.c_void_p, C.c_int32, C.c_float, C.c_size_t
        L.btx_moe_sizes.argtypes = [C.POINTER(MoeDesc), C.POINTER(sz), C.POINTER(sz)]
        L.btx_moe_forward.argtypes = [C.POINTER(MoeDesc), vp, vp, vp, vp, vp, vp, vp, vp, C.POINTER(RoutingOut), vp, vp,
                                      sz, vp]
        L.btx_moe_backward.argtypes = [C.POINTER(MoeDesc), vp, vp, vp, vp, vp, vp, vp, vp, f32, vp, vp, vp, vp, vp, vp,
                                       vp, vp, i32, vp, sz, vp]
        L.btx_moe_step_host.argtypes = [C.POINTER(MoeDesc)] + [vp] * 15 + [f32] + [vp] * 5 + [i32, vp, vp, sz, vp, vp]
        L.btx_set_stage_events.argtypes = [C.POINTER(vp), i32]
        L.btx_selftest_wait_expiry.argtypes = [vp, sz, vp]
        L.btx_lb_loss_workspace_size.argtypes = [C.POINTER(MoeDesc), C.POINTER(sz)]
        L.btx_lb_loss.argtypes = [C.POINTER(MoeDesc), vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.btx_lb_loss_noalloc.argtypes = [C.POINTER(MoeDesc), vp, vp, vp, vp, vp, vp, vp]
        L.btx_merge_workspace_size.argtypes = [i32, C.c_uint64, C.POINTER(sz)]
        L.btx_merge.argtypes = [i32, i32, C.POINTER(MergeItem), C.c_uint64, vp, sz, vp]
        L.btx_merge_ffn_workspace_size.argtypes = [i32, i32, C.POINTER(sz)]
        L.btx_merge_ffn.argtypes = [i32, i32, i32, i32, i32, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp, vp, vp,
                                    vp, sz, vp]
        L.btx_device_status.argtypes = [vp, vp, C.POINTER(i32)]
        L.btx_status_string.argtypes = [i32]
        L.btx_status_string.restype = C.c_char_p
        L.btx_version.restype = i32
        for name in EXPORTS:
            if name not in ("btx_status_string", "btx_version"):
                getattr(L, name).restype = i32
        _lib = L
    return _lib


def _dtype_code(t) -> int:
    if t == torch.float32:
        return BTX_F32
    if t == torch.bfloat16:
        return BTX_BF16
    raise TypeError(f"unsupported dtype {t}")


def _ptr(t):
    if t is None:
        return None
    if not t.is_cuda:
        raise RuntimeError("btx: tensors must live on a CUDA device (there is no CPU path)")
    if not t.is_contiguous():
        raise RuntimeError("btx: tensors must be contiguous")
    return C.c_void_p(t.data_ptr())


def _stream(device):
    return C.c_void_p(torch.cuda.current_stream(device).cuda_stream)


def _on(device):
    """The library works on the current device (its helper stream, multiprocessor count and static scratch
    are looked up per current device): every call runs with the tensors' device made current."""
    if torch.device(device).type != "cuda":
        raise RuntimeError("btx: tensors must live on a CUDA device (there is no CPU path)")
    return torch.cuda.device(device)


def make_desc(T, d_model, d_ff, E, k, dtype, routing=ROUTE_TOPK, lb_alpha=0.01, lb_stopgrad_u=False,
              save_for_backward=False, skip_wgrad=False, gumbel_tau=0.0, capacity_factor=0.0) -> MoeDesc:
    code = _dtype_code(dtype) if isinstance(dtype, torch.dtype) else int(dtype)
    return MoeDesc(T, d_model, d_ff, E, k, code, routing, lb_alpha, int(lb_stopgrad_u), int(save_for_backward),
                   int(skip_wgrad), float(gumbel_tau), float(capacity_factor))


def btx_moe_sizes(desc: MoeDesc):
    ws, sv = C.c_size_t(0), C.c_size_t(0)
    s = lib().btx_moe_sizes(C.byref(desc), C.byref(ws), C.byref(sv))
    if s != BTX_OK:
        raise BtxError(s, "btx_moe_sizes")
    return ws.value, sv.value


@dataclass
class Routing:
    logits: torch.Tensor
    topk_idx: torch.Tensor
    gates: torch.Tensor
    probs: torch.Tensor
    counts: torch.Tensor
    offsets: torch.Tensor
    perm: torch.Tensor
    inv_perm: torch.Tensor
    u: torch.Tensor
    p: torch.Tensor
    lb_loss: torch.Tensor

    @staticmethod
    def empty(desc: MoeDesc, device):
        k = desc.E if desc.routing == ROUTE_SOFT else desc.k
        T, E, R = desc.T, desc.E, desc.T * k
        f = dict(dtype=torch.float32, device=device)
        i = dict(dtype=torch.int32, device=device)
        return Routing(torch.empty((T, E), **f), torch.empty((T, k), **i), torch.empty((T, k), **f),
                       torch.empty((T, E), **f), torch.empty(E, **i), torch.empty(E + 1, **i), torch.empty(R, **i),
                       torch.empty(R, **i), torch.empty(E, **f), torch.empty(E, **f), torch.empty(1, **f))

    def as_struct(self) -> RoutingOut:
        return RoutingOut(*[t.data_ptr() for t in (self.logits, self.topk_idx, self.gates, self.probs, self.counts,
                                                   self.offsets, self.perm, self.inv_perm, self.u, self.p,
                                                   self.lb_loss)])


def alloc_buffers(desc: MoeDesc, device):
    """(workspace, saved) byte tensors of the sizes btx_moe_sizes reports."""
    ws, sv = btx_moe_sizes(desc)
    return (torch.empty(ws, dtype=torch.uint8, device=device),
            torch.empty(max(sv, 16), dtype=torch.uint8, device=device))


def btx_moe_forward(desc, x, w_router, router_bias, w1, w3, w2, y, routing, saved, workspace, router_noise=None):
    ro = routing.as_struct() if routing is not None else None
    with _on(x.device):
        s = lib().btx_moe_forward(C.byref(desc), _ptr(x), _ptr(w_router), _ptr(router_bias), _ptr(router_noise),
                                  _ptr(w1), _ptr(w3), _ptr(w2),
                                  _ptr(y), C.byref(ro) if ro is not None else None, _ptr(saved), _ptr(workspace),
                                  workspace.numel(), _stream(x.device))
    if s != BTX_OK:
        raise BtxError(s, "btx_moe_forward")


def btx_moe_backward(desc, x, w_router, router_bias, w1, w3, w2, dy, lb_grad_scale, saved, dx, dw_router, dbias,
                     dw1, dw3, dw2, accumulate, workspace, router_noise=None, dlogits=None):
    with _on(x.device):
        s = lib().btx_moe_backward(C.byref(desc), _ptr(x), _ptr(w_router), _ptr(router_bias), _ptr(router_noise),
                                   _ptr(w1), _ptr(w3), _ptr(w2),
                                   _ptr(dy), float(lb_grad_scale), _ptr(saved), _ptr(dx), _ptr(dw_router), _ptr(dbias),
                                   _ptr(dlogits), _ptr(dw1), _ptr(dw3), _ptr(dw2), int(accumulate), _ptr(workspace),
                                   workspace.numel(), _stream(x.device))
    if s != BTX_OK:
        raise BtxError(s, "btx_moe_backward")


def btx_moe_step_host(desc, x_host, dy_host, y_host, dx_host, loss_host, x_dev, dy_dev, y_dev, dx_dev, w_router,
                      router_bias, w1, w3, w2, lb_grad_scale, dw_router, dbias, dw1, dw3, dw2, accumulate, saved,
                      workspace, router_noise=None, copy_stream=None):
    """Forward + backward with activations in (pinned) host tensors; see btx.h.  `copy_stream` is an
    optional torch.cuda.Stream on which the dy upload and the y download overlap the compute."""
    for t in (x_host, dy_host, y_host, dx_host, loss_host):
        if t.is_cuda or not t.is_contiguous():
            raise RuntimeError("btx_moe_step_host: host tensors must be contiguous CPU tensors")
    hp = lambda t: C.c_void_p(t.data_ptr())
    with _on(x_dev.device):
        s = lib().btx_moe_step_host(C.byref(desc), hp(x_host), hp(dy_host), hp(y_host), hp(dx_host), hp(loss_host),
                                    _ptr(x_dev), _ptr(dy_dev), _ptr(y_dev), _ptr(dx_dev), _ptr(w_router),
                                    _ptr(router_bias), _ptr(router_noise), _ptr(w1), _ptr(w3), _ptr(w2),
                                    float(lb_grad_scale),
                                    _ptr(dw_router), _ptr(dbias), _ptr(dw1), _ptr(dw3), _ptr(dw2), int(accumulate),
                                    _ptr(saved), _ptr(workspace), workspace.numel(), _stream(x_dev.device),
                                    C.c_void_p(copy_stream.cuda_stream) if copy_stream is not None else None)
    if s != BTX_OK:
        raise BtxError(s, "btx_moe_step_host")


_stage_keepalive = None


def btx_set_stage_events(events):
    """events: list of torch.cuda.Event(enable_timing=True) that have been recorded at least once
    (so that their handles exist), or None to switch the hook off."""
    global _stage_keepalive
    if events is None:
        _stage_keepalive = None
        s = lib().btx_set_stage_events(None, 0)
    else:
        arr = (C.c_void_p * len(events))(*[e.cuda_event for e in events])
        _stage_keepalive = (arr, events)
        s = lib().btx_set_stage_events(arr, len(events))
    if s != BTX_OK:
        raise BtxError(s, "btx_set_stage_events")


def btx_lb_loss_workspace_size(desc):
    sz = C.c_size_t(0)
    s = lib().btx_lb_loss_workspace_size(C.byref(desc), C.byref(sz))
    if s != BTX_OK:
        raise BtxError(s, "btx_lb_loss_workspace_size")
    return sz.value


def btx_lb_loss(desc, logits, loss, u, p, dlogits, workspace, router_bias=None):
    with _on(logits.device):
        s = lib().btx_lb_loss(C.byref(desc), _ptr(logits), _ptr(router_bias), _ptr(loss), _ptr(u), _ptr(p),
                              _ptr(dlogits), _ptr(workspace), workspace.numel(), _stream(logits.device))
    if s != BTX_OK:
        raise BtxError(s, "btx_lb_loss")


def btx_lb_loss_noalloc(desc, logits, loss, u, p, dlogits, router_bias=None):
    """btx_lb_loss on the library's own static scratch: no workspace argument, nothing allocated."""
    with _on(logits.device):
        s = lib().btx_lb_loss_noalloc(C.byref(desc), _ptr(logits), _ptr(router_bias), _ptr(loss), _ptr(u), _ptr(p),
                                      _ptr(dlogits), _stream(logits.device))
    if s != BTX_OK:
        raise BtxError(s, "btx_lb_loss_noalloc")


def btx_merge_workspace_size(n_models, n_items):
    sz = C.c_size_t(0)
    s = lib().btx_merge_workspace_size(n_models, n_items, C.byref(sz))
    if s != BTX_OK:
        raise BtxError(s, "btx_merge_workspace_size")
    return sz.value


def btx_merge(models, outputs, workspace=None):
    """models: list of N dicts name -> tensor; outputs: dict name -> tensor ([N, ...] for names
    containing '.ffn.', same shape as the sources otherwise).  Builds the item table and calls
    the library once; returns the workspace (keep it alive until the stream has run)."""
    n = len(models)
    names = list(models[0].keys())
    items = (MergeItem * len(names))()
    keep = []
    dtype = None
    for i, name in enumerate(names):
        srcs = [m[name] for m in models]
        dtype = srcs[0].dtype
        arr = (C.c_void_p * n)(*[_ptr(s).value for s in srcs])
        keep.append(arr)
        items[i].kind = PARAM_FFN if ".ffn." in name else PARAM_AVERAGE
        items[i].layer = 0
        items[i].numel = srcs[0].numel()
        items[i].src = C.cast(arr, C.POINTER(C.c_void_p))
        items[i].dst = _ptr(outputs[name]).value
    device = models[0][names[0]].device
    if workspace is None:
        workspace = torch.empty(btx_merge_workspace_size(n, len(names)), dtype=torch.uint8, device=device)
    with _on(device):
        s = lib().btx_merge(n, _dtype_code(dtype), items, len(names), _ptr(workspace), workspace.numel(),
                            _stream(device))
    if s != BTX_OK:
        raise BtxError(s, "btx_merge")
    return workspace


def btx_merge_ffn(w1s, w3s, w2s, layout, chunks, w1_dst, w3_dst, w2_dst, workspace=None):
    """One layer's FFN matrices of N models (lists of [F,d], [F,d], [d,F] tensors) into expert tensors in
    the STACK, SPLIT or BLEND layout; see btx.h."""
    n = len(w1s)
    F, d = w1s[0].shape
    arr = lambda ts: (C.c_void_p * n)(*[_ptr(t).value for t in ts])
    a1, a3, a2 = arr(w1s), arr(w3s), arr(w2s)
    device = w1s[0].device
    if workspace is None:
        sz = C.c_size_t(0)
        s = lib().btx_merge_ffn_workspace_size(n, max(1, chunks), C.byref(sz))
        if s != BTX_OK:
            raise BtxError(s, "btx_merge_ffn_workspace_size")
        workspace = torch.empty(sz.value, dtype=torch.uint8, device=device)
    with _on(device):
        s = lib().btx_merge_ffn(n, _dtype_code(w1s[0].dtype), layout, chunks, d, F, a1, a3, a2, _ptr(w1_dst),
                                _ptr(w3_dst), _ptr(w2_dst), _ptr(workspace), workspace.numel(), _stream(device))
    if s != BTX_OK:
        raise BtxError(s, "btx_merge_ffn")
    return workspace


def btx_selftest_wait_expiry(workspace):
    """Makes one bounded device-side wait run out on purpose; see btx.h."""
    with _on(workspace.device):
        s = lib().btx_selftest_wait_expiry(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _stream(workspace.device))
    if s != BTX_OK:
        raise BtxError(s, "btx_selftest_wait_expiry")


def btx_device_status(workspace):
    st = C.c_int32(0)
    with _on(workspace.device):
        s = lib().btx_device_status(_ptr(workspace), _stream(workspace.device), C.byref(st))
    if s != BTX_OK:
        raise BtxError(s, "btx_device_status")
    return st.value
