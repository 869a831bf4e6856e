"""Parity at the benchmark's full sizes (Llama-2-7B-shaped layer: d_model 4096, d_ff 11008, 4 experts),
in the launch configuration bench.py times.  Routing, counts and the permutation are compared in full
and bit-exactly (oracle fed the GPU's fp32 logits); floating-point outputs are compared on sampled
tokens (y, dx) and sampled hidden units (dW1, dW3, dW2), which the oracle computes one by one; the router
gradient is compared in full (all E x d entries) through the oracle's sum over the GPU's d(loss)/d(logits),
which itself is compared on the sampled tokens; plus properties that hold at any size (router-gradient
rows sum to zero)."""
import numpy as np
import pytest
import torch

from oracle import btx_oracle as o
from paper_2403_07816_b200 import binding as B
from paper_2403_07816_b200 import synth
from util import gpu_backward, gpu_forward, np64, rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
D, F, E = 4096, 11008, 4
TOL = 1e-2
ALPHA = 0.01


def full_size_case(T, k, seed, routing=B.ROUTE_TOPK, bias=None, backward=True, n_tok=192, n_hidden=24, F=F, E=E,
                   capacity_factor=0.0):
    inp = synth.moe_inputs(T, D, F, E, seed, torch.bfloat16, DEV, with_dy=backward)
    fwd = gpu_forward(inp, k, routing, ALPHA, bias, save=backward, capacity_factor=capacity_factor)
    r = fwd["routing"]
    kk = E if routing == B.ROUTE_SOFT else k
    cpu = {n: np64(t) for n, t in inp.items()}
    b64 = None if bias is None else np64(bias)
    rng = np.random.default_rng(seed)
    tok = np.sort(rng.choice(T, size=min(n_tok, T), replace=False))

    # routing: full size, bit-exact on the GPU's logits
    z_gpu = r.logits.cpu().numpy()
    assert rel_err(z_gpu, o.router_logits(cpu["x"], cpu["w_router"], b64)) <= TOL
    z, idx, g, p_tok = o.route(cpu["x"], cpu["w_router"], kk, routing, b64, logits=z_gpu)
    assert np.array_equal(r.topk_idx.cpu().numpy(), idx)
    keep = o.capacity_keep(idx, E, o.expert_capacity(T, kk, E, capacity_factor)) if capacity_factor > 0 else None
    counts, offsets, perm, inv_perm = o.dispatch(idx, E, keep)
    for name, want in [("counts", counts), ("offsets", offsets), ("perm", perm), ("inv_perm", inv_perm)]:
        assert np.array_equal(getattr(r, name).cpu().numpy(), want), name
    assert rel_err(r.gates.cpu().numpy(), g) <= 1e-5 and rel_err(r.probs.cpu().numpy(), p_tok) <= 1e-5
    loss, u, p = o.lb_loss(o.dense_gates(idx, g, E), p_tok, ALPHA)
    assert abs(r.lb_loss.item() - loss) <= 1e-5 * loss
    assert rel_err(r.u.cpu().numpy(), u) <= 1e-5 and rel_err(r.p.cpu().numpy(), p) <= 1e-5

    # y on sampled tokens
    ref = o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], kk, routing, ALPHA,
                        router_bias=b64, logits=z_gpu, tokens=tok, capacity_factor=capacity_factor)
    y = np64(fwd["y"])
    assert np.all(np.isfinite(y))
    e_y = np.max(np.abs(y[tok] - ref["y"])) / np.max(np.abs(ref["y"]))
    assert e_y <= TOL, f"y {e_y}"
    if keep is not None and kk == 1:
        dropped = torch.from_numpy(~keep[:, 0]).to(DEV)
        assert float(fwd["y"][dropped].abs().max()) == 0.0                # a dropped token's output is exactly 0
    if not backward:
        return counts
    got = gpu_backward(inp, fwd, 1.0, bias)
    sl = o.moe_backward_token_slice(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], cpu["dy"], idx, g,
                                    p_tok, u, p, tok, routing, ALPHA, 1.0, False, keep=keep)
    dx = np64(got["dx"])
    assert np.all(np.isfinite(dx))
    e_dx = np.max(np.abs(dx[tok] - sl["dx"])) / np.max(np.abs(sl["dx"]))
    assert e_dx <= TOL, f"dx {e_dx}"
    # weight gradients on sampled hidden units, over all tokens of the expert
    for e in range(E):
        J = np.sort(rng.choice(F, size=n_hidden, replace=False))
        d1, d3, d2 = o.expert_wgrad_hidden_slice(cpu["x"], cpu["w1"], cpu["w3"], cpu["w2"], cpu["dy"], idx, g, e, J,
                                                 keep=keep)
        Jt = torch.from_numpy(J).to(DEV)
        for name, want, have in [("dw1", d1, got["dw1"][e][Jt]), ("dw3", d3, got["dw3"][e][Jt]),
                                 ("dw2", d2, got["dw2"][e][:, Jt])]:
            if np.max(np.abs(want)) == 0:
                assert float(have.abs().max()) == 0.0
                continue
            err = rel_err(np64(have), want)
            assert err <= TOL, f"{name}[{e}] {err}"
    # router gradient at full size.  d(loss)/d(logits) on the sampled tokens against the oracle; then dW_l and
    # dbias over ALL tokens against the oracle's sums of the GPU's own dz (x and dz are the same numbers on both
    # sides, so only the order of the fp32 additions differs: a far tighter bar than the layer's tolerance).
    dz_gpu = got["dlogits"].cpu().numpy()
    assert np.all(np.isfinite(dz_gpu))
    e_dz = np.max(np.abs(dz_gpu[tok] - sl["dlogits"])) / np.max(np.abs(sl["dlogits"]))
    assert e_dz <= TOL, f"dlogits {e_dz}"
    dwr_ref, db_ref = o.router_wgrad_from_dz(cpu["x"], dz_gpu)
    e_dwr = rel_err(np64(got["dw_router"]), dwr_ref)
    assert e_dwr <= 1e-4, f"dw_router {e_dwr}"
    summed = float(np.max(np.sum(np.abs(dz_gpu.astype(np.float64)), axis=0)))
    e_db = float(np.max(np.abs(np64(got["dbias"]) - db_ref))) / summed
    assert e_db <= 1e-4, f"dbias {e_db}"
    # properties at full size: every softmax Jacobian is shift invariant
    dwr = np64(got["dw_router"])
    assert np.all(np.isfinite(dwr))
    assert np.max(np.abs(dwr.sum(axis=0))) <= 1e-3 * np.max(np.abs(dwr))
    assert abs(np64(got["dbias"]).sum()) <= 1e-3 * np.max(np.abs(np64(got["dbias"]))) + 1e-6
    for n in ("dw1", "dw3", "dw2"):
        assert bool(torch.isfinite(got[n]).all()), n
    return counts


def test_forward_T4096_seed1():
    full_size_case(4096, 2, seed=1, backward=False)


def test_forward_backward_T16384_seed2():
    counts = full_size_case(16384, 2, seed=2, n_tok=256, n_hidden=64)
    assert counts.min() > 0.2 * 32768 and counts.max() < 0.3 * 32768      # roughly uniform loads


def test_switch_top1_T16384_seed3():
    full_size_case(16384, 1, seed=3, routing=B.ROUTE_SWITCH, n_tok=128, n_hidden=16)


def test_soft_routing_T16384_seed3():
    full_size_case(16384, 4, seed=3, routing=B.ROUTE_SOFT, n_tok=96, n_hidden=12)


def test_skewed_top2_T16384_seed3():
    bias = synth.skew_bias(E, DEV)
    counts = full_size_case(16384, 2, seed=3, bias=bias, n_tok=128, n_hidden=16)
    assert counts[0] > 0.4 * 32768                                        # expert 0 takes the largest share


def test_switch_capacity_factor_T16384_seed7():
    # Section 4.1: Switch routing with capacity factor 1.5; the skewed router overflows expert 0,
    # whose later tokens are dropped
    bias = synth.skew_bias(E, DEV)
    counts = full_size_case(16384, 1, seed=7, routing=B.ROUTE_SWITCH, bias=bias, n_tok=128, n_hidden=16,
                            capacity_factor=1.5)
    assert counts[0] == 6144 and counts.sum() < 16384


def test_top2_capacity_factor_T4096_seed8():
    bias = synth.skew_bias(E, DEV)
    counts = full_size_case(4096, 2, seed=8, bias=bias, n_tok=96, n_hidden=12, capacity_factor=1.25)
    assert counts[0] == 2560 and counts.sum() < 8192


def test_split_expert_shapes_E8():
    # "Splitting experts" (Section 3.3): each FFN cut into two chunks of d_ff/2 gives 8 modules;
    # the paper trains top-4 of 8; top-2 of 8 exercises sparser loads
    full_size_case(4096, 4, seed=5, F=5504, E=8, n_tok=96, n_hidden=12)
    full_size_case(4096, 2, seed=6, F=5504, E=8, n_tok=96, n_hidden=12)


def test_decode_shaped_T32_two_layers_seed4():
    for layer in range(2):
        inp = synth.moe_inputs(32, D, F, E, 4, torch.bfloat16, DEV, layer=layer, with_dy=False)
        fwd = gpu_forward(inp, 2, save=False)
        cpu = {n: np64(t) for n, t in inp.items()}
        z_gpu = fwd["routing"].logits.cpu().numpy()
        ref = o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], 2, alpha=ALPHA, logits=z_gpu)
        assert np.array_equal(fwd["routing"].topk_idx.cpu().numpy(), ref["topk_idx"])
        assert np.array_equal(fwd["routing"].perm.cpu().numpy(), ref["perm"])
        assert rel_err(np64(fwd["y"]), ref["y"]) <= TOL


@pytest.mark.parametrize("T,F_,E_,k,routing,cf", [
    (48, 5504, 8, 2, B.ROUTE_TOPK, 0.0),       # split experts, top-2 of 8: MMA N = 48, eight experts streamed
    (64, 11008, 4, 1, B.ROUTE_SWITCH, 1.0),    # the widest token tile (N = 64), Switch gate, capacity limit with drops
    (9, 11008, 4, 4, B.ROUTE_SOFT, 0.0),       # every expert for every token, N = 16 with 9 real tokens
])
def test_decode_shaped_variants_full_width(T, F_, E_, k, routing, cf):
    """The one-kernel inference forward at d = 4096 and the full hidden widths, in the launch configuration the
    decode bench uses (74 CTA pairs, several tiles per pair): the whole output against the oracle."""
    inp = synth.moe_inputs(T, D, F_, E_, 7, torch.bfloat16, DEV, with_dy=False)
    bias = synth.skew_bias(E_, DEV) if cf > 0 else None
    fwd = gpu_forward(inp, k, routing, ALPHA, bias, save=False, capacity_factor=cf)
    cpu = {n: np64(t) for n, t in inp.items()}
    z_gpu = fwd["routing"].logits.cpu().numpy()
    kk = E_ if routing == B.ROUTE_SOFT else k
    ref = o.moe_forward(cpu["x"], cpu["w_router"], cpu["w1"], cpu["w3"], cpu["w2"], kk, routing, ALPHA,
                        router_bias=None if bias is None else np64(bias), logits=z_gpu, capacity_factor=cf)
    r = fwd["routing"]
    for name in ("topk_idx", "counts", "offsets", "perm", "inv_perm"):
        assert np.array_equal(getattr(r, name).cpu().numpy(), ref[name]), name
    if cf > 0:
        assert not ref["keep"].all()
    assert rel_err(r.gates.cpu().numpy(), ref["gates"]) <= TOL
    assert abs(float(r.lb_loss.item()) - ref["lb_loss"]) <= TOL * max(abs(ref["lb_loss"]), 1e-30)
    assert rel_err(np64(fwd["y"]), ref["y"]) <= TOL


def test_merge_llama2_7b_shaped_tensors_seed4():
    """MiX merge at the sizes of the Llama-2-7B shape (Section 3.2): two layers plus embeddings, head and final
    norm of four BF16 parameter sets (5.4 GB read).  Averaged tensors against the fp64 mean rounded once;
    stacked feed-forward slots bit for bit, compared on the device."""
    models = synth.expert_models(4, 2, D, F, 32000, seed=4, dtype=torch.bfloat16, device=DEV)
    out = {}
    for n, t in models[0].items():
        out[n] = torch.empty(((4,) + tuple(t.shape)) if ".ffn." in n else tuple(t.shape), dtype=torch.bfloat16, device=DEV)
    B.btx_merge(models, out)
    torch.cuda.synchronize()
    for n in out:
        if ".ffn." in n:
            for m in range(4):
                assert torch.equal(out[n][m], models[m][n]), (n, m)
            continue
        if out[n].numel() > (1 << 24):
            # the two [32000, 4096] tensors: 2048 sampled rows through the oracle, and on the device every
            # element between the smallest and the largest of its four sources
            rows = torch.from_numpy(np.sort(np.random.default_rng(4).choice(out[n].shape[0], 2048, replace=False))).to(DEV)
            stack = torch.stack([m[n] for m in models]).float()
            assert bool(((out[n].float() >= stack.amin(0)) & (out[n].float() <= stack.amax(0))).all()), n
            del stack
            srcs = [np64(m[n][rows]) for m in models]
            got = np64(out[n][rows])
        else:
            srcs = [np64(m[n]) for m in models]
            got = np64(out[n])
        mean = o.merge_mean(srcs)
        # The kernel sums in fp32 in model order (three roundings of at most 2^-24 of a partial sum) and rounds
        # once to bf16: the result lies within half a bf16 ulp of the exact mean's binade plus that fp32 error.
        # (Where the exact mean sits that close to a rounding boundary the stored value may be the other
        # neighbour, one ulp from the oracle's rounding; both are within the bound.)
        mean_abs = sum(np.abs(a) for a in srcs) / 4
        half_ulp = np.exp2(np.floor(np.log2(np.maximum(np.abs(mean), 2.0 ** -126))) - 8.0)
        assert np.all(np.abs(got - mean) <= half_ulp * (1 + 1e-9) + 3 * 2.0 ** -24 * mean_abs), n
        assert np.mean(got != o.merge_average(srcs, "bf16")) < 1e-3, n
        del srcs, mean, got
