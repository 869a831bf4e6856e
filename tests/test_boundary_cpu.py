"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments before touching the device."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2403_07816_b200 import binding as B
from paper_2403_07816_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    builder.build()
    return B.lib()


def header_functions():
    text = open(os.path.join(ROOT, "include", "btx.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(btx_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = header_functions()
    assert len(names) >= 9
    for n in names:
        assert hasattr(L, n), n
    assert sorted(B.EXPORTS) == names          # the binding wraps exactly the declared calls


def test_version_and_status_strings(L):
    assert L.btx_version() >= 100
    seen = {L.btx_status_string(i).decode() for i in range(7)}
    assert len(seen) == 7 and "ok" in seen


def test_sizes_and_argument_validation(L):
    d = B.make_desc(256, 256, 688, 4, 2, torch.float32, save_for_backward=True)
    ws, sv = B.btx_moe_sizes(d)
    assert ws > 0 and sv > 0 and ws % 256 == 0
    bigger = B.make_desc(512, 256, 688, 4, 2, torch.float32, save_for_backward=True)
    assert B.btx_moe_sizes(bigger)[0] > ws
    bad = [B.make_desc(0, 256, 688, 4, 2, torch.float32),            # T < 1
           B.make_desc(8, 256, 688, 4, 5, torch.float32),            # k > E
           B.make_desc(8, 256, 688, 4, 0, torch.float32),            # k < 1
           B.make_desc(8, 256, 688, 4, 2, torch.float32, routing=B.ROUTE_SWITCH),   # Switch needs k = 1
           B.make_desc(8, 256, 688, 4, 2, 7)]                        # unknown dtype
    for desc in bad:
        with pytest.raises(B.BtxError) as ei:
            B.btx_moe_sizes(desc)
        assert ei.value.status == 1
    for desc in [B.make_desc(8, 250, 688, 4, 2, torch.bfloat16),     # d not a multiple of 8
                 B.make_desc(8, 256, 688, 65, 2, torch.float32)]:    # more than 64 experts
        with pytest.raises(B.BtxError) as ei:
            B.btx_moe_sizes(desc)
        assert ei.value.status == 2
    B.btx_moe_sizes(B.make_desc(8, 256, 688, 64, 2, torch.float32))  # 64 experts are covered
    # Sample Top-1: one expert, defined without the load-balancing loss
    B.btx_moe_sizes(B.make_desc(8, 256, 688, 4, 1, torch.float32, routing=B.ROUTE_SAMPLE1, lb_alpha=0.0, gumbel_tau=0.5))
    with pytest.raises(B.BtxError) as ei:
        B.btx_moe_sizes(B.make_desc(8, 256, 688, 4, 1, torch.float32, routing=B.ROUTE_SAMPLE1, lb_alpha=0.01))
    assert ei.value.status == 2
    with pytest.raises(B.BtxError) as ei:
        B.btx_moe_sizes(B.make_desc(8, 256, 688, 4, 2, torch.float32, routing=B.ROUTE_SAMPLE1, lb_alpha=0.0))
    assert ei.value.status == 1
    # soft routing ignores k
    B.btx_moe_sizes(B.make_desc(8, 256, 688, 4, 0, torch.float32, routing=B.ROUTE_SOFT))
    # capacity factor: non-negative, and meaningless when every expert takes every token
    B.btx_moe_sizes(B.make_desc(8, 256, 688, 4, 1, torch.float32, routing=B.ROUTE_SWITCH, capacity_factor=1.5))
    for desc in [B.make_desc(8, 256, 688, 4, 1, torch.float32, routing=B.ROUTE_SWITCH, capacity_factor=-1.0),
                 B.make_desc(8, 256, 688, 4, 1, torch.float32, capacity_factor=float("nan")),
                 B.make_desc(8, 256, 688, 4, 4, torch.float32, routing=B.ROUTE_SOFT, capacity_factor=1.5)]:
        with pytest.raises(B.BtxError) as ei:
            B.btx_moe_sizes(desc)
        assert ei.value.status == 1


def test_null_and_misaligned_pointers_rejected_before_any_launch(L):
    d = B.make_desc(8, 64, 64, 4, 2, torch.float32)
    vp = C.c_void_p
    s = L.btx_moe_forward(C.byref(d), None, None, None, None, None, None, None, None, None, None, None, 0, None)
    assert s == 1
    a = vp(4096)
    s = L.btx_moe_forward(C.byref(d), vp(4100), a, None, None, a, a, a, a, None, None, a, 1 << 40, None)
    assert s == 1                                        # x not 16-byte aligned
    s = L.btx_moe_forward(C.byref(d), a, a, None, None, a, a, a, a, None, None, a, 16, None)
    assert s == 3                                        # workspace too small
    s = L.btx_moe_backward(C.byref(d), a, a, None, None, a, a, a, a, 1.0, None, a, a, None, None, a, a, a, 0, a, 1 << 40,
                           None)
    assert s == 1                                        # saved missing
    s = L.btx_moe_backward(C.byref(d), a, a, None, None, a, a, a, a, 1.0, a, a, a, None, vp(4100), a, a, a, 0, a,
                           1 << 40, None)
    assert s == 1                                        # dlogits not 16-byte aligned
    sz = C.c_size_t(0)
    assert L.btx_merge_workspace_size(0, 3, C.byref(sz)) == 1
    assert L.btx_merge_workspace_size(4, 3, C.byref(sz)) == 0 and sz.value > 0
    assert L.btx_merge(99, 0, None, 1, a, 1 << 20, None) == 2
    assert L.btx_merge(4, 0, None, 0, None, 0, None) == 0    # nothing to do


def test_refused_calls_return_before_touching_the_device(L):
    """Every argument check precedes the first CUDA call: a refused request comes back with its own status
    (on a host without a GPU any CUDA call would have turned it into BTX_ERR_CUDA or BTX_ERR_ARCH)."""
    vp = C.c_void_p
    a = vp(4096)
    big = 1 << 40
    sample1 = B.make_desc(8, 0, 0, 4, 1, torch.float32, routing=B.ROUTE_SAMPLE1, lb_alpha=0.0, gumbel_tau=0.5)
    assert L.btx_lb_loss(C.byref(sample1), a, None, a, a, a, None, a, big, None) == 2
    assert L.btx_lb_loss_noalloc(C.byref(sample1), a, None, a, a, a, None, None) == 2
    ok = B.make_desc(8, 0, 0, 4, 2, torch.float32)
    assert L.btx_lb_loss(C.byref(ok), None, None, a, a, a, None, a, big, None) == 1       # logits missing
    assert L.btx_lb_loss(C.byref(ok), a, None, a, a, a, None, a, 16, None) == 3           # workspace too small
    huge = B.make_desc(1 << 20, 0, 0, 8, 2, torch.float32)
    assert L.btx_lb_loss_noalloc(C.byref(huge), a, None, a, a, a, None, None) == 3        # beyond the static scratch
    assert L.btx_selftest_wait_expiry(a, 16, None) == 3
    assert L.btx_device_status(None, None, None) == 1
    d = B.make_desc(8, 64, 64, 4, 2, torch.float32, save_for_backward=True)
    assert L.btx_moe_step_host(C.byref(d), *([None] * 15), 1.0, *([None] * 5), 0, None, None, 0, None, None) == 1


def test_synthetic_model_shapes_match_the_pinned_table():
    """The merge workload's shape table (the input generator's copy) is the one the oracle's copy pins to the
    paper's Table 4 parameter counts."""
    from oracle import btx_oracle as o
    from paper_2403_07816_b200 import synth
    for args in [(32, 4096, 11008, 32000), (2, 256, 688, 1024)]:
        assert synth.llama_like_param_shapes(*args) == o.llama_like_param_shapes(*args)


def test_binding_refuses_cpu_tensors(L):
    d = B.make_desc(8, 64, 64, 4, 2, torch.float32)
    x = torch.zeros(8, 64)
    with pytest.raises(RuntimeError, match="CUDA device"):
        B.btx_moe_forward(d, x, x, None, x, x, x, x, None, None, x)
