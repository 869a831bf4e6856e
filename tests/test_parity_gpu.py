"""Parity of the CUDA path (through the C ABI) against the CPU oracle, element by element, on
seeded inputs.  Routing and the dispatch permutation must be bit-exact when the oracle is fed the
GPU's fp32 logits; floating-point outputs must satisfy max|err|/max|ref| <= 1e-5 in FP32 mode and
<= 1e-2 in BF16 mode."""
import numpy as np
import pytest
import torch

from oracle import btx_oracle as o
from paper_2403_07816_b200 import binding as B
from paper_2403_07816_b200 import synth
from util import TOL, check_backward, check_forward, gpu_backward, gpu_forward, np64, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

DTYPES = [torch.float32, torch.bfloat16]
IDS = ["f32", "bf16"]


def run_case(T, d, F, E, k, dtype, seed, routing=B.ROUTE_TOPK, alpha=0.01, bias=None, lb_scale=1.0,
             stopgrad_u=False, backward=True):
    inp = synth.moe_inputs(T, d, F, E, seed, dtype, DEV)
    tol = TOL[dtype]
    kk = E if routing == B.ROUTE_SOFT else k
    fwd = gpu_forward(inp, k, routing, alpha, bias, save=backward, stopgrad_u=stopgrad_u)
    cpu, b64, z_gpu, ref = check_forward(inp, fwd, kk, routing, alpha, bias, tol)
    if backward:
        got = gpu_backward(inp, fwd, lb_scale, bias)
        check_backward(cpu, b64, z_gpu, got, kk, routing, alpha, lb_scale, stopgrad_u, tol)
    return inp, fwd, ref


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_tiny_config_forward_backward(dtype):
    # T=256, d=256, F=688 (= 5*128 + 48: ragged column tiles), E=4, top-2, alpha = 0.01, seed 0
    run_case(256, 256, 688, 4, 2, dtype, seed=0)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
@pytest.mark.parametrize("T,d,F,E,k", [(37, 64, 72, 5, 3), (1, 128, 128, 4, 2), (300, 136, 264, 8, 2),
                                        (129, 64, 64, 1, 1), (515, 192, 328, 3, 1),
                                        (700, 64, 72, 4, 2)])      # T*k > 1024: multi-block routing kernels
def test_ragged_shapes(dtype, T, d, F, E, k):
    run_case(T, d, F, E, k, dtype, seed=11, alpha=0.05, lb_scale=0.7)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
@pytest.mark.parametrize("E", [32, 64])
@pytest.mark.parametrize("T,d,F,routing,k", [(200, 72, 40, B.ROUTE_TOPK, 8), (150, 64, 72, B.ROUTE_SOFT, 0),
                                             (40, 8, 8, B.ROUTE_TOPK, 0), (2500, 64, 64, B.ROUTE_SWITCH, 1),
                                             (300, 64, 72, B.ROUTE_TOPK, 3), (12, 64, 72, B.ROUTE_TOPK, 3)])
def test_maximum_expert_count_and_smallest_widths(dtype, E, T, d, F, routing, k):
    """E = 64 (the library's limit) and E = 32 (one warp lane per expert exactly): sparse loads with experts
    that receive nothing, every expert selected (k = 0 stands for k = E), rows of a single 16-byte vector,
    more padded row tiles than tokens, and the small-batch path with more row tiles than its usual handful."""
    run_case(T, d, F, E, k if k else E, dtype, seed=17, routing=routing, alpha=0.05, lb_scale=0.7)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_switch_routing(dtype):
    run_case(200, 128, 136, 4, 1, dtype, seed=3, routing=B.ROUTE_SWITCH, alpha=0.02)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_soft_routing(dtype):
    run_case(150, 128, 136, 4, 4, dtype, seed=3, routing=B.ROUTE_SOFT, alpha=0.02)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_router_bias_skew_and_empty_expert(dtype):
    bias = torch.tensor([1.5, 0.0, -100.0, 0.2], dtype=torch.float32, device=DEV)   # expert 2 never chosen
    inp, fwd, ref = run_case(260, 128, 200, 4, 2, dtype, seed=5, bias=bias)
    assert int(fwd["routing"].counts[2].item()) == 0
    assert int(fwd["routing"].counts[0].item()) > 130


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_lb_stopgrad_and_zero_alpha(dtype):
    run_case(96, 64, 72, 4, 2, dtype, seed=6, alpha=0.3, stopgrad_u=True)
    run_case(96, 64, 72, 4, 2, dtype, seed=6, alpha=0.0)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_accumulate_adds_to_existing_gradients(dtype):
    inp = synth.moe_inputs(70, 64, 72, 4, 8, dtype, DEV)
    fwd = gpu_forward(inp, 2)
    cpu, b64, z_gpu, _ = check_forward(inp, fwd, 2, B.ROUTE_TOPK, 0.01, None, TOL[dtype])
    got = gpu_backward(inp, fwd, accumulate=True, init=0.25)
    check_backward(cpu, b64, z_gpu, got, 2, B.ROUTE_TOPK, 0.01, 1.0, False, TOL[dtype], base=0.25)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_tied_logits_go_to_lower_index_and_identical_experts(dtype):
    # zero router: every logit ties -> experts (0, 1), gates 1/2, L_LB = alpha exactly;
    # identical experts -> the layer equals the dense FFN
    inp = synth.moe_inputs(64, 64, 72, 4, 9, dtype, DEV)
    inp["w_router"].zero_()
    for n in ("w1", "w3", "w2"):
        inp[n][1:] = inp[n][:1]
    fwd = gpu_forward(inp, 2, alpha=0.01, save=False)
    r = fwd["routing"]
    assert (r.topk_idx.cpu().numpy() == np.array([[0, 1]])).all()
    assert (r.gates.cpu().numpy() == 0.5).all()
    assert abs(float(r.lb_loss.item()) - 0.01) < 1e-8
    dense = o.swiglu_ffn(np64(inp["x"]), np64(inp["w1"][0]), np64(inp["w3"][0]), np64(inp["w2"][0]))
    assert rel_err(np64(fwd["y"]), dense) <= TOL[dtype]


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_frozen_experts_skip_weight_gradients(dtype):
    # the paper's freeze ablation: only dx and the router gradients are produced
    for T in (96, 700):                                   # small-batch and multi-block routing paths
        inp = synth.moe_inputs(T, 64, 72, 4, 12, dtype, DEV)
        fwd = gpu_forward(inp, 2, alpha=0.05, skip_wgrad=True)
        cpu, b64, z_gpu, _ = check_forward(inp, fwd, 2, B.ROUTE_TOPK, 0.05, None, TOL[dtype])
        got = gpu_backward(inp, fwd)
        assert got["dw1"] is None
        check_backward(cpu, b64, z_gpu, got, 2, B.ROUTE_TOPK, 0.05, 1.0, False, TOL[dtype])


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
@pytest.mark.parametrize("tau", [0.7, 0.0], ids=["soft", "hard"])
def test_sample_top1_routing(dtype, tau):
    # Gumbel noise is an input; tau > 0: gate = largest entry of SoftMax((z+G)/tau); tau = 0: hard sample, gate 1
    for T in (96, 700):
        inp = synth.moe_inputs(T, 64, 72, 4, 13, dtype, DEV)
        noise = synth.gumbel_noise(T, 4, 13, DEV)
        fwd = gpu_forward(inp, 1, B.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=tau)
        cpu, b64, z_gpu, ref = check_forward(inp, fwd, 1, B.ROUTE_SAMPLE1, 0.0, None, TOL[dtype], noise=noise, tau=tau)
        if tau == 0.0:
            assert bool((fwd["routing"].gates == 1.0).all())
        got = gpu_backward(inp, fwd)
        check_backward(cpu, b64, z_gpu, got, 1, B.ROUTE_SAMPLE1, 0.0, 1.0, False, TOL[dtype], noise=noise, tau=tau)
        if tau == 0.0:
            assert float(got["dw_router"].abs().max()) == 0.0


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
@pytest.mark.parametrize("tau", [0.7, 0.0], ids=["soft", "hard"])
def test_sample_top1_perturbed_logits_that_tie_in_fp32(dtype, tau):
    """The expert of Sample Top-1 is decided on z + G formed by one fp32 addition: where two sums differ only
    below fp32 resolution they tie and the lower index wins, whatever the temperature (which scales only the
    softmax).  Tokens are unit vectors, so the logits are router weights exactly."""
    for T in (64, 700):                                   # one-launch and multi-block routing kernels
        inp = synth.moe_inputs(T, 64, 72, 4, 14, dtype, DEV)
        inp["x"].zero_()
        inp["x"][:, 0] = 1.0
        inp["w_router"].zero_()
        inp["w_router"][:, 0] = torch.tensor([0.0, 2.0 ** -25, -3.0, -3.0], dtype=dtype, device=DEV)
        noise = torch.zeros(T, 4, dtype=torch.float32, device=DEV)
        noise[:, 0] = 1.0
        noise[:, 1] = 1.0                                  # fp64: expert 1 leads by 2^-25; fp32: 1 + 2^-25 == 1
        noise[T // 2:, 1] = 1.0 + 2.0 ** -20               # second half: expert 1 leads in fp32 as well
        fwd = gpu_forward(inp, 1, B.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=tau)
        idx = fwd["routing"].topk_idx.cpu().numpy()[:, 0]
        assert (idx[:T // 2] == 0).all() and (idx[T // 2:] == 1).all()
        cpu, b64, z_gpu, ref = check_forward(inp, fwd, 1, B.ROUTE_SAMPLE1, 0.0, None, TOL[dtype], noise=noise, tau=tau)
        got = gpu_backward(inp, fwd)
        check_backward(cpu, b64, z_gpu, got, 1, B.ROUTE_SAMPLE1, 0.0, 1.0, False, TOL[dtype], noise=noise, tau=tau)


def test_results_are_deterministic_across_runs():
    inp = synth.moe_inputs(256, 256, 688, 4, 0, torch.float32, DEV)
    a = gpu_forward(inp, 2)
    ga = gpu_backward(inp, a)
    b = gpu_forward(inp, 2)
    gb = gpu_backward(inp, b)
    assert torch.equal(a["y"], b["y"])
    for n in ga:
        assert torch.equal(ga[n], gb[n]), n


@pytest.mark.parametrize("with_bias", [False, True], ids=["nobias", "bias"])
@pytest.mark.parametrize("routing,k", [(B.ROUTE_TOPK, 2), (B.ROUTE_SWITCH, 1), (B.ROUTE_SOFT, 4)])
def test_lb_loss_entry_point(routing, k, with_bias):
    T, E, alpha = 333, 4, 0.01
    g = torch.Generator(device="cpu").manual_seed(4)
    logits = (torch.randn(T, E, generator=g) * 1.3).to(DEV)
    bias = torch.tensor([0.75, -0.5, 0.0, 1.25], device=DEV) if with_bias else None
    desc = B.make_desc(T, 0, 0, E, k, torch.float32, routing, alpha)
    ws = torch.empty(B.btx_lb_loss_workspace_size(desc), dtype=torch.uint8, device=DEV)
    loss = torch.empty(1, device=DEV); u = torch.empty(E, device=DEV); p = torch.empty(E, device=DEV)
    dz = torch.empty(T, E, device=DEV)
    B.btx_lb_loss(desc, logits, loss, u, p, dz, ws, router_bias=bias)
    z = (logits + bias).cpu().numpy() if with_bias else logits.cpu().numpy()    # the same fp32 sum the kernel forms
    kk = E if routing == B.ROUTE_SOFT else k
    want, wu, wp = o.lb_loss_from_logits(z, kk, routing, alpha)
    assert abs(loss.item() - want) <= 1e-5 * want
    assert rel_err(u.cpu().numpy(), wu) <= 1e-5 and rel_err(p.cpu().numpy(), wp) <= 1e-5
    assert rel_err(dz.cpu().numpy(), o.lb_loss_grad(z, kk, routing, alpha)) <= 1e-5


@pytest.mark.parametrize("dtype,name", [(torch.float32, "f32"), (torch.bfloat16, "bf16")], ids=IDS)
def test_merge_toy_models(dtype, name):
    # 4 seeded copies of a 2-layer d=256 toy model (vocab 1024) merged into one MoE model
    models = synth.expert_models(4, 2, 256, 688, 1024, seed=0, dtype=dtype, device=DEV)
    # one tensor with an odd element count exercises the scalar tail
    for m, mod in enumerate(models):
        mod["odd_tail"] = synth.normal((1003,), 0.02, 0, 999, dtype, DEV, layer=m)
    out = {}
    for n, t in models[0].items():
        out[n] = torch.full(((4,) + tuple(t.shape)) if ".ffn." in n else tuple(t.shape), 7.0, dtype=dtype, device=DEV)
    B.btx_merge(models, out)
    torch.cuda.synchronize()
    cpu_models = [{n: np64(t) for n, t in m.items()} for m in models]
    ref = o.merge_models(cpu_models, name)
    ulp = 2.0 ** -8 if dtype == torch.bfloat16 else 2.0 ** -24
    for n in out:
        got = np64(out[n])
        if ".ffn." in n:
            assert np.array_equal(got, ref[n]), n                  # copies are bit-exact
        else:
            # The kernel sums in fp32 in model order: each of the N-1 additions rounds by at most
            # 2^-24 of a partial sum (<= sum |src|); the store rounds once more to the storage type.
            mean_abs = sum(np.abs(m[n]) for m in cpu_models) / len(cpu_models)
            bound = ulp * np.abs(ref[n]) * 1.0001 + 3 * 2.0 ** -24 * mean_abs + 1e-45
            assert np.all(np.abs(got - ref[n]) <= bound), n
            assert rel_err(got, ref[n]) <= TOL[dtype]
            if dtype == torch.bfloat16:
                assert np.mean(got != ref[n]) < 1e-2, n            # the fp32 sum rarely flips a bf16 rounding
    # identical models: the merge returns the seed bit for bit (N = 4 is a power of two)
    same = [models[0]] * 4
    B.btx_merge(same, out)
    torch.cuda.synchronize()
    for n in out:
        if ".ffn." not in n:
            assert torch.equal(out[n], models[0][n]), n


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_merge_split_and_blend_layouts(dtype):
    N, F, d = 4, 704, 256            # F/4 = 176 hidden units: whole 16-byte vectors in both dtypes
    w1s = [synth.normal((F, d), 0.02, 7, 10 + i, dtype, DEV) for i in range(N)]
    w3s = [synth.normal((F, d), 0.02, 7, 20 + i, dtype, DEV) for i in range(N)]
    w2s = [synth.normal((d, F), 0.02, 7, 30 + i, dtype, DEV) for i in range(N)]
    cpu = [[np64(t) for t in ts] for ts in (w1s, w3s, w2s)]
    for layout, chunks in [(B.FFN_STACK, 1), (B.FFN_SPLIT, 2), (B.FFN_SPLIT, 4), (B.FFN_BLEND, 0)]:
        ref = o.merge_ffn_layout(cpu[0], cpu[1], cpu[2], layout, chunks)
        outs = [torch.full(r.shape, 3.0, dtype=dtype, device=DEV) for r in ref]
        B.btx_merge_ffn(w1s, w3s, w2s, layout, chunks, *outs)
        torch.cuda.synchronize()
        for got, want in zip(outs, ref):
            assert np.array_equal(np64(got), want), (layout, chunks)       # pure copies: bit-exact


@pytest.mark.gpu
@pytest.mark.parametrize("overlap", [False, True], ids=["one_stream", "copy_stream"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16], ids=["f32", "bf16"])
def test_step_host_matches_oracle(dtype, overlap):
    """The host-buffer entry point (pinned x, dy in; y, dx, loss out), with and without a second
    stream for the copies, gives the oracle's y, dx, loss and weight gradients."""
    dev = torch.device(DEV)
    T, d, F, E, k = 777, 128, 328, 4, 2
    inp = synth.moe_inputs(T, d, F, E, 41, dtype, DEV)
    desc = B.make_desc(T, d, F, E, k, dtype, B.ROUTE_TOPK, 0.01, False, True)
    ws, saved = B.alloc_buffers(desc, dev)
    hx, hdy = inp["x"].cpu().pin_memory(), inp["dy"].cpu().pin_memory()
    hy, hdx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
    hloss = torch.zeros(1, dtype=torch.float32).pin_memory()
    xd, dyd, yd, dxd = (torch.empty_like(inp["x"]) for _ in range(4))
    f32 = dict(dtype=torch.float32, device=dev)
    out = dict(dw_router=torch.empty(E, d, **f32), dbias=torch.empty(E, **f32), dw1=torch.empty(E, F, d, **f32),
               dw3=torch.empty(E, F, d, **f32), dw2=torch.empty(E, d, F, **f32))
    cs = torch.cuda.Stream(device=dev) if overlap else None
    for _ in range(2):       # the second call reuses every buffer: the copy stream must be joined back
        hy.zero_(); hdx.zero_()
        B.btx_moe_step_host(desc, hx, hdy, hy, hdx, hloss, xd, dyd, yd, dxd, inp["w_router"], None, inp["w1"],
                            inp["w3"], inp["w2"], 1.0, out["dw_router"], out["dbias"], out["dw1"], out["dw3"],
                            out["dw2"], 0, saved, ws, copy_stream=cs)
        torch.cuda.current_stream(dev).synchronize()
        assert B.btx_device_status(ws) == B.BTX_OK
    tol = TOL[dtype]
    cpu = {n: np64(t) for n, t in inp.items()}
    # routing decisions are taken on the GPU's fp32 logits (the same kernel, run through the device entry point)
    z_ref = gpu_forward(inp, k, save=False)["routing"].logits.cpu().numpy()
    fwd = o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], k, B.ROUTE_TOPK, 0.01,
                        logits=z_ref)
    assert rel_err(np64(hy), fwd["y"]) <= tol
    assert abs(float(hloss.item()) - fwd["lb_loss"]) <= tol * abs(fwd["lb_loss"])
    got = dict(out, dx=hdx)
    check_backward(cpu, None, z_ref, got, k, B.ROUTE_TOPK, 0.01, 1.0, False, tol)
    assert torch.equal(yd.cpu(), hy) and torch.equal(dxd.cpu(), hdx)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
@pytest.mark.parametrize("routing,k,cf", [(B.ROUTE_SWITCH, 1, 1.5), (B.ROUTE_SWITCH, 1, 0.5), (B.ROUTE_TOPK, 2, 0.75),
                                          (B.ROUTE_TOPK, 1, 1.0)])
def test_capacity_factor_drops_tokens(dtype, routing, k, cf):
    """Expert capacity with token dropping (Section 4.1): kept rows, permutation and drop marks
    bit-exact; y, dx and every gradient within tolerance; a skewed router makes expert 0 overflow."""
    T, d, F, E = 1500, 128, 328, 4
    inp = synth.moe_inputs(T, d, F, E, 51, dtype, DEV)
    bias = synth.skew_bias(E, DEV)
    tol = TOL[dtype]
    fwd = gpu_forward(inp, k, routing, 0.01, bias, capacity_factor=cf)
    cpu, b64, z_gpu, ref = check_forward(inp, fwd, k, routing, 0.01, bias, tol, capacity_factor=cf)
    assert not ref["keep"].all() and (fwd["routing"].inv_perm.cpu().numpy() < 0).sum() == (~ref["keep"]).sum()
    got = gpu_backward(inp, fwd, 1.0, bias)
    check_backward(cpu, b64, z_gpu, got, k, routing, 0.01, 1.0, False, tol, capacity_factor=cf)


@pytest.mark.parametrize("dtype", DTYPES, ids=IDS)
def test_capacity_factor_small_batch_and_limits(dtype):
    """The small-batch path (one-launch routing, weight-streaming expert kernels) under a limit; a limit nobody reaches changes
    nothing; SOFT routing with a limit is refused."""
    T, d, F, E, k = 120, 256, 512, 4, 2         # T*k <= 64*E: the weight-streaming expert kernels run
    inp = synth.moe_inputs(T, d, F, E, 52, dtype, DEV)
    bias = synth.skew_bias(E, DEV)
    tol = TOL[dtype]
    fwd = gpu_forward(inp, k, B.ROUTE_TOPK, 0.01, bias, capacity_factor=0.75)
    cpu, b64, z_gpu, ref = check_forward(inp, fwd, k, B.ROUTE_TOPK, 0.01, bias, tol, capacity_factor=0.75)
    assert not ref["keep"].all()
    got = gpu_backward(inp, fwd, 1.0, bias)
    check_backward(cpu, b64, z_gpu, got, k, B.ROUTE_TOPK, 0.01, 1.0, False, tol, capacity_factor=0.75)
    free = gpu_forward(inp, k, B.ROUTE_TOPK, 0.01, bias)
    wide = gpu_forward(inp, k, B.ROUTE_TOPK, 0.01, bias, capacity_factor=float(E))
    assert torch.equal(free["y"], wide["y"]) and torch.equal(free["routing"].perm, wide["routing"].perm)
    with pytest.raises(B.BtxError):
        gpu_forward(inp, E, B.ROUTE_SOFT, 0.01, None, capacity_factor=1.5)


@pytest.mark.parametrize("T,d,F,E,k,routing,cf", [
    (32, 256, 688, 4, 2, B.ROUTE_TOPK, 0.0),      # the decode shape in small: F = 5*128 + 48, one 32-column group
    (5, 128, 136, 4, 2, B.ROUTE_TOPK, 0.0),       # N = 16 with 5 real tokens; the second CTA's token rows are all padding
    (64, 264, 392, 4, 2, B.ROUTE_TOPK, 0.0),      # N = 64: both column groups; contraction tails in both passes
    (33, 128, 256, 8, 8, B.ROUTE_SOFT, 0.0),      # every expert for every token; N = 48
    (17, 192, 328, 2, 1, B.ROUTE_SWITCH, 0.0),
    (1, 128, 128, 1, 1, B.ROUTE_TOPK, 0.0),       # a single token, a single expert
    (40, 128, 264, 4, 2, B.ROUTE_TOPK, 0.5),      # capacity limit: dropped assignments are skipped in pass 2
    (48, 64, 72, 3, 1, B.ROUTE_SAMPLE1, 0.0),
    (64, 64, 72, 64, 8, B.ROUTE_TOPK, 0.0),       # the expert limit: two experts per lane in the selection, 64 small experts
    (40, 72, 40, 33, 33, B.ROUTE_SOFT, 0.0),      # one expert beyond a warp's lanes, every expert for every token
    (64, 128, 136, 5, 2, B.ROUTE_TOPK, 0.4),      # tight capacity at N = 64: most assignments dropped
])
def test_inference_forward_of_a_few_tokens(T, d, F, E, k, routing, cf):
    """BF16 forward that keeps nothing for backward, at most 64 tokens: every expert's weights meet all tokens
    (no gather, SwiGLU formed in the first kernel's epilogue, routing beside it).  Compared with the oracle in
    full, with the forward that saves for backward (other kernels: same routing bits, y within tolerance), and
    run twice on one workspace (the second call finds the first call's scratch and status word)."""
    dtype = torch.bfloat16
    inp = synth.moe_inputs(T, d, F, E, 61, dtype, DEV)
    bias = synth.normal((E,), 0.3, 61, 77, torch.float32, DEV)
    noise = synth.gumbel_noise(T, E, 61, DEV) if routing == B.ROUTE_SAMPLE1 else None
    alpha = 0.0 if routing == B.ROUTE_SAMPLE1 else 0.02
    kk = E if routing == B.ROUTE_SOFT else k
    fwd = gpu_forward(inp, k, routing, alpha, bias, save=False, noise=noise, tau=0.8, capacity_factor=cf)
    check_forward(inp, fwd, kk, routing, alpha, bias, TOL[dtype], noise=noise, tau=0.8, capacity_factor=cf)
    kept = gpu_forward(inp, k, routing, alpha, bias, save=True, noise=noise, tau=0.8, capacity_factor=cf)
    for name in ("logits", "topk_idx", "gates", "probs", "perm", "inv_perm", "counts", "u", "p", "lb_loss"):
        assert torch.equal(getattr(fwd["routing"], name), getattr(kept["routing"], name)), name
    assert rel_err(np64(fwd["y"]), np64(kept["y"])) <= TOL[dtype]
    y1 = fwd["y"].clone()
    r = fwd["routing"]
    B.btx_moe_forward(fwd["desc"], inp["x"], inp["w_router"], bias, inp["w1"], inp["w3"], inp["w2"], fwd["y"], r, None,
                      fwd["ws"], router_noise=noise)
    assert B.btx_device_status(fwd["ws"]) == B.BTX_OK
    assert torch.equal(fwd["y"], y1)


def test_bounded_wait_expires_and_the_context_stays_usable():
    """The safety net of the tensor-core kernels: a device-side wait that nothing will satisfy gives up
    after its limit, the status word reports it, the kernel returns, and later calls work as usual."""
    ws = torch.empty(4096, dtype=torch.uint8, device=DEV)
    B.btx_selftest_wait_expiry(ws)
    assert B.btx_device_status(ws) == B.BTX_ERR_TIMEOUT
    run_case(300, 128, 264, 4, 2, torch.bfloat16, seed=3)        # same context, fresh call: status OK inside


def test_training_step_replays_from_a_cuda_graph():
    """Forward + backward issue only stream-ordered work (kernels, memsets, event fork/join with the
    library's helper stream), so the pair can be captured once and replayed: same bits as the direct calls."""
    T, d, F, E, k = 1200, 256, 528, 4, 2
    inp = synth.moe_inputs(T, d, F, E, 23, torch.bfloat16, DEV)
    desc = B.make_desc(T, d, F, E, k, torch.bfloat16, B.ROUTE_TOPK, 0.01, False, True)
    ws, saved = B.alloc_buffers(desc, DEV)
    f32 = dict(dtype=torch.float32, device=DEV)
    outs = dict(y=torch.empty_like(inp["x"]), dx=torch.empty_like(inp["x"]), dwr=torch.empty(E, d, **f32),
                dbias=torch.empty(E, **f32), dw1=torch.empty(E, F, d, **f32), dw3=torch.empty(E, F, d, **f32),
                dw2=torch.empty(E, d, F, **f32))

    def step():
        B.btx_moe_forward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], outs["y"], None,
                          saved, ws)
        B.btx_moe_backward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], inp["dy"], 1.0,
                           saved, outs["dx"], outs["dwr"], outs["dbias"], outs["dw1"], outs["dw3"], outs["dw2"], 0, ws)

    step()
    torch.cuda.synchronize()
    direct = {n: t.clone() for n, t in outs.items()}
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                   # warm-up on the capture stream
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for t in outs.values():
        t.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert B.btx_device_status(ws) == B.BTX_OK
    for n, t in outs.items():
        assert torch.equal(t, direct[n]), n


def test_inference_forward_replays_from_a_cuda_graph():
    """The one-kernel forward of a few tokens is a single cooperative launch; three layers of it can be captured
    once and replayed, with the direct calls' bits."""
    T, d, F, E, k = 32, 1024, 2048, 4, 2
    sets = [synth.moe_inputs(T, d, F, E, 4, torch.bfloat16, DEV, layer=l, with_dy=False) for l in range(3)]
    desc = B.make_desc(T, d, F, E, k, torch.bfloat16, B.ROUTE_TOPK, 0.01, False, False)
    ws, _ = B.alloc_buffers(desc, DEV)
    ys = [torch.empty(T, d, dtype=torch.bfloat16, device=DEV) for _ in sets]

    def step():
        for inp, y in zip(sets, ys):
            B.btx_moe_forward(desc, inp["x"], inp["w_router"], None, inp["w1"], inp["w3"], inp["w2"], y, None, None, ws)

    step()
    torch.cuda.synchronize()
    direct = [y.clone() for y in ys]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for y in ys:
        y.zero_()
    graph.replay()
    graph.replay()
    torch.cuda.synchronize()
    assert B.btx_device_status(ws) == B.BTX_OK
    for got, want in zip(ys, direct):
        assert torch.equal(got, want)
