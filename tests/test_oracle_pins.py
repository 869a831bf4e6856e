"""Pins for the CPU oracle: closed forms, invariants, brute force, finite differences and the
paper's printed parameter counts.  None of these call the CUDA path."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import btx_oracle as o

RNG = np.random.default_rng


def small_problem(seed, T=24, d=12, F=20, E=4, scale_r=1.0):
    r = RNG(seed)
    x = r.standard_normal((T, d))
    wr = r.standard_normal((E, d)) * scale_r
    w1 = r.standard_normal((E, F, d)) * 0.3
    w3 = r.standard_normal((E, F, d)) * 0.3
    w2 = r.standard_normal((E, d, F)) * 0.3
    dy = r.standard_normal((T, d))
    return x, wr, w1, w3, w2, dy


# ---- scalar re-statement used for brute force on tiny inputs ---------------------------------

def scalar_ffn(xv, W1, W3, W2):
    F, d = len(W1), len(xv)
    a = []
    for f in range(F):
        h1 = sum(W1[f][c] * xv[c] for c in range(d))
        h3 = sum(W3[f][c] * xv[c] for c in range(d))
        a.append(h1 / (1.0 + math.exp(-h1)) * h3)
    return [sum(W2[c][f] * a[f] for f in range(F)) for c in range(d)]


def scalar_moe_token(xv, Wr, W1, W3, W2, k):
    """Enumerate every k-subset; keep the one with the largest logit sum (lowest indices on a
    tie); mix the experts of that subset with a softmax restricted to it."""
    E, d = len(Wr), len(xv)
    z = [sum(Wr[i][c] * xv[c] for c in range(d)) for i in range(E)]
    best = None
    for S in itertools.combinations(range(E), k):          # lexicographic = lowest indices first
        s = sum(z[i] for i in S)
        if best is None or s > best[0]:
            best = (s, S)
    S = best[1]
    den = sum(math.exp(z[i]) for i in S)
    y = [0.0] * d
    for i in S:
        gi = math.exp(z[i]) / den
        yi = scalar_ffn(xv, W1[i], W3[i], W2[i])
        for c in range(d):
            y[c] += gi * yi[c]
    return set(S), y


# ---- closed forms -----------------------------------------------------------------------------

def test_worked_example_closed_form():
    # one token, d = 1, two experts; logits (ln 3, 0) -> gates (3/4, 1/4)
    x = np.array([[1.0]])
    wr = np.array([[math.log(3.0)], [0.0]])
    w1 = np.array([[[1.0]], [[0.0]]])
    w3 = np.array([[[2.0]], [[5.0]]])
    w2 = np.array([[[1.0]], [[7.0]]])
    out = o.moe_forward(x, wr, w1, w3, w2, k=2, alpha=0.01)
    np.testing.assert_allclose(out["gates"], [[0.75, 0.25]], rtol=1e-14)
    assert out["topk_idx"].tolist() == [[0, 1]]
    # expert 0: silu(1)*2 = 2/(1+e^-1); expert 1: silu(0) = 0
    np.testing.assert_allclose(out["y"], [[0.75 * 2.0 / (1.0 + math.exp(-1.0))]], rtol=1e-14)
    # u = (3/4, 1/4) = p  ->  L = 0.01 * 2 * (9/16 + 1/16)
    np.testing.assert_allclose(out["lb_loss"], 0.01 * 2 * (10.0 / 16.0), rtol=1e-14)


def test_operand_orientation_non_square():
    # W1, W3 are [F, d] and W2 is [d, F]: with F != d a transposed operand cannot even multiply,
    # and a swapped W1/W3 changes the value below.
    x = np.array([[1.0, 2.0]])
    w1 = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])        # h1 = (1, 2, 3)
    w3 = np.array([[1.0, 1.0], [0.0, 0.5], [2.0, 0.0]])        # h3 = (3, 1, 2)
    w2 = np.array([[1.0, 0.0, 1.0], [0.0, 2.0, -1.0]])
    silu = lambda v: v / (1.0 + math.exp(-v))
    a = [silu(1.0) * 3.0, silu(2.0) * 1.0, silu(3.0) * 2.0]
    want = [a[0] + a[2], 2.0 * a[1] - a[2]]
    np.testing.assert_allclose(o.swiglu_ffn(x, w1, w3, w2), [want], rtol=1e-14)


def test_lb_loss_closed_forms():
    ln3 = math.log(3.0)
    # two tokens preferring different experts, top-1 of 2 (gate of a lone selected logit is 1)
    z = np.array([[ln3, 0.0], [0.0, ln3]])
    loss, u, p = o.lb_loss_from_logits(z, 1, o.ROUTE_TOPK, 0.01)
    np.testing.assert_allclose(u, [0.5, 0.5]); np.testing.assert_allclose(p, [0.5, 0.5])
    np.testing.assert_allclose(loss, 0.01, rtol=1e-14)
    # both prefer expert 0: u = (1, 0), p = (3/4, 1/4): L = alpha * 2 * 3/4
    z = np.array([[ln3, 0.0], [ln3, 0.0]])
    loss, u, p = o.lb_loss_from_logits(z, 1, o.ROUTE_TOPK, 0.01)
    np.testing.assert_allclose(loss, 0.015, rtol=1e-14)
    # Switch gate is the full-softmax probability: u = (3/4, 0): L = alpha * 2 * 9/16
    loss, u, p = o.lb_loss_from_logits(z, 1, o.ROUTE_SWITCH, 0.01)
    np.testing.assert_allclose(u, [0.75, 0.0])
    np.testing.assert_allclose(loss, 0.01 * 2 * 9.0 / 16.0, rtol=1e-14)


def test_zero_router_ties_and_uniform_loss():
    x, wr, w1, w3, w2, _ = small_problem(1)
    for k in (1, 2, 3):
        out = o.moe_forward(x, wr * 0.0, w1, w3, w2, k=k, alpha=0.01)
        assert (out["topk_idx"] == np.arange(k)[None, :]).all()          # ties -> lowest indices in order
        np.testing.assert_allclose(out["gates"], 1.0 / k)
        np.testing.assert_allclose(out["probs"], 0.25)
        np.testing.assert_allclose(out["lb_loss"], 0.01, rtol=1e-14)    # alpha * E * sum u_i / E
    # signed zeros tie as well
    z = np.array([[0.0, -0.0, 0.0, -0.0], [-0.0, 0.0, -0.0, 0.0]])
    assert o.top_k_select(z, 2).tolist() == [[0, 1], [0, 1]]


def test_dominant_expert_loss_tends_to_alpha_E():
    z = np.tile(np.array([[40.0, 0.0, 0.0, 0.0]]), (5, 1))
    loss, u, p = o.lb_loss_from_logits(z, 1, o.ROUTE_TOPK, 0.01)
    np.testing.assert_allclose(loss, 0.04, rtol=1e-12)


# ---- invariants -------------------------------------------------------------------------------

@pytest.mark.parametrize("routing,k", [(o.ROUTE_TOPK, 1), (o.ROUTE_TOPK, 2), (o.ROUTE_TOPK, 3), (o.ROUTE_SOFT, 4)])
def test_identical_experts_reduce_to_dense_ffn(routing, k):
    x, wr, w1, w3, w2, _ = small_problem(2)
    w1 = np.repeat(w1[:1], 4, axis=0); w3 = np.repeat(w3[:1], 4, axis=0); w2 = np.repeat(w2[:1], 4, axis=0)
    out = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing)
    np.testing.assert_allclose(out["y"], o.swiglu_ffn(x, w1[0], w3[0], w2[0]), rtol=1e-12, atol=1e-14)


def test_single_expert_is_dense_ffn():
    x, wr, w1, w3, w2, _ = small_problem(3, E=1)
    out = o.moe_forward(x, wr, w1, w3, w2, k=1, alpha=0.01)
    np.testing.assert_allclose(out["y"], o.swiglu_ffn(x, w1[0], w3[0], w2[0]), rtol=1e-13)
    np.testing.assert_allclose(out["lb_loss"], 0.01, rtol=1e-14)


def test_sparse_evaluation_equals_literal_sum_over_all_experts():
    x, wr, w1, w3, w2, _ = small_problem(4)
    for routing, k in [(o.ROUTE_TOPK, 2), (o.ROUTE_SWITCH, 1), (o.ROUTE_SOFT, 4)]:
        a = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing)["y"]
        b = o.moe_forward_all_experts(x, wr, w1, w3, w2, k=k, routing=routing)
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


def test_expert_relabelling():
    x, wr, w1, w3, w2, dy = small_problem(5)
    sigma = np.array([2, 0, 3, 1])                       # new expert j is old expert sigma[j]
    a = o.moe_forward(x, wr, w1, w3, w2, k=2)
    b = o.moe_forward(x, wr[sigma], w1[sigma], w3[sigma], w2[sigma], k=2)
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(a["lb_loss"], b["lb_loss"], rtol=1e-13)
    assert (sigma[b["topk_idx"]] == a["topk_idx"]).all()
    ga = o.moe_backward(x, wr, w1, w3, w2, dy, k=2)
    gb = o.moe_backward(x, wr[sigma], w1[sigma], w3[sigma], w2[sigma], dy, k=2)
    np.testing.assert_allclose(ga["dx"], gb["dx"], rtol=1e-11, atol=1e-13)
    for name in ("dw1", "dw3", "dw2", "dw_router"):
        np.testing.assert_allclose(ga[name][sigma], gb[name], rtol=1e-11, atol=1e-13)


@pytest.mark.parametrize("E,k", [(2, 1), (4, 2), (5, 3), (6, 2)])
def test_brute_force_subsets(E, k):
    r = RNG(10 + E)
    T, d, F = 6, 3, 4
    x = r.standard_normal((T, d)); wr = r.standard_normal((E, d))
    w1 = r.standard_normal((E, F, d)); w3 = r.standard_normal((E, F, d)); w2 = r.standard_normal((E, d, F))
    out = o.moe_forward(x, wr, w1, w3, w2, k=k)
    for t in range(T):
        S, y = scalar_moe_token(x[t].tolist(), wr.tolist(), w1.tolist(), w3.tolist(), w2.tolist(), k)
        assert set(out["topk_idx"][t].tolist()) == S
        np.testing.assert_allclose(out["y"][t], y, rtol=1e-12, atol=1e-13)
        # slots are ordered by decreasing logit
        zs = out["logits"][t][out["topk_idx"][t]]
        assert (np.diff(zs) <= 0).all()


def test_gate_equivalences():
    r = RNG(6)
    z = r.standard_normal((50, 4)) * 2
    idx = o.top_k_select(z, 2)
    g = o.gate_values(z, idx, o.ROUTE_TOPK)
    p = o.full_softmax(z)
    psel = np.take_along_axis(p, idx.astype(np.int64), axis=1)
    np.testing.assert_allclose(g, psel / psel.sum(1, keepdims=True), rtol=1e-13)   # renormalised full softmax
    idx4 = o.top_k_select(z, 4)
    g4 = o.gate_values(z, idx4, o.ROUTE_SOFT)
    np.testing.assert_allclose(o.dense_gates(idx4, g4, 4), p, rtol=1e-13)          # soft = top-E
    idx1 = o.top_k_select(z, 1)
    gs = o.gate_values(z, idx1, o.ROUTE_SWITCH)
    np.testing.assert_allclose(gs[:, 0], p.max(axis=1), rtol=1e-13)                 # Switch gate
    assert (idx1[:, 0] == np.argmax(p, axis=1)).all()
    # softmax is shift invariant
    np.testing.assert_allclose(o.full_softmax(z + 3.0), p, rtol=1e-12)


def test_forward_bookkeeping():
    x, wr, w1, w3, w2, _ = small_problem(7, T=40)
    out = o.moe_forward(x, wr, w1, w3, w2, k=2)
    np.testing.assert_allclose(out["gates"].sum(1), 1.0, rtol=1e-14)
    np.testing.assert_allclose(out["u"].sum(), 1.0, rtol=1e-13)
    np.testing.assert_allclose(out["p"].sum(), 1.0, rtol=1e-13)
    counts, offsets, perm, inv = out["counts"], out["offsets"], out["perm"], out["inv_perm"]
    assert counts.sum() == 80 and offsets[0] == 0 and offsets[-1] == 80
    assert (np.diff(offsets) == counts).all()
    assert (perm[inv] == np.arange(80)).all() and (inv[perm] == np.arange(80)).all()
    flat = out["topk_idx"].reshape(-1)
    for e in range(4):
        rows = perm[offsets[e]:offsets[e + 1]]
        assert (flat[rows] == e).all()
        assert (np.diff(rows // 2) > 0).all()             # strictly increasing token index
    # a hand-checked dispatch
    idx = np.array([[1, 0], [0, 2], [1, 2]], dtype=np.int32)
    c, off, pm, iv = o.dispatch(idx, 3)
    assert c.tolist() == [2, 2, 2] and off.tolist() == [0, 2, 4, 6]
    assert pm.tolist() == [1, 2, 0, 4, 3, 5] and iv.tolist() == [2, 0, 1, 4, 3, 5]


# ---- gradients --------------------------------------------------------------------------------

def total_loss(x, wr, w1, w3, w2, G, k, routing, alpha, lam, bias=None):
    out = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=alpha, router_bias=bias)
    return float(np.sum(out["y"] * G)) + lam * out["lb_loss"]


@pytest.mark.parametrize("routing,k", [(o.ROUTE_TOPK, 2), (o.ROUTE_TOPK, 1), (o.ROUTE_SWITCH, 1), (o.ROUTE_SOFT, 4)])
def test_gradients_against_finite_differences(routing, k):
    x, wr, w1, w3, w2, G = small_problem(8, T=10, d=6, F=7, E=4, scale_r=1.5)
    bias = np.array([0.1, -0.2, 0.0, 0.3])
    alpha, lam = 0.7, 1.3                     # large alpha so the loss terms are visible
    # the point must be far from a routing boundary
    z = o.router_logits(x, wr, bias)
    zs = np.sort(z, axis=1)
    assert np.min(np.diff(zs, axis=1)) > 1e-3
    g = o.moe_backward(x, wr, w1, w3, w2, G, k=k, routing=routing, alpha=alpha, lb_grad_scale=lam,
                       router_bias=bias)
    r = RNG(99)
    h = 1e-6
    params = dict(x=x, wr=wr, w1=w1, w3=w3, w2=w2, bias=bias)
    names = dict(x="dx", wr="dw_router", w1="dw1", w3="dw3", w2="dw2", bias="dbias")
    for pname, arr in params.items():
        for _ in range(6):
            pos = tuple(int(r.integers(0, s)) for s in arr.shape)
            old = arr[pos]
            arr[pos] = old + h
            lp = total_loss(x, wr, w1, w3, w2, G, k, routing, alpha, lam, bias)
            arr[pos] = old - h
            lm = total_loss(x, wr, w1, w3, w2, G, k, routing, alpha, lam, bias)
            arr[pos] = old
            fd = (lp - lm) / (2 * h)
            an = g[names[pname]][pos]
            assert abs(fd - an) <= 2e-6 * max(1.0, abs(fd)), (pname, pos, fd, an)


def test_lb_gradient_alone_and_stopgrad():
    r = RNG(11)
    z = r.standard_normal((12, 4)) * 1.5
    alpha = 0.5
    for routing, k in [(o.ROUTE_TOPK, 2), (o.ROUTE_SWITCH, 1), (o.ROUTE_SOFT, 4)]:
        dz = o.lb_loss_grad(z, k, routing, alpha)
        h = 1e-6
        for _ in range(8):
            pos = (int(r.integers(0, 12)), int(r.integers(0, 4)))
            zp = z.copy(); zp[pos] += h
            zm = z.copy(); zm[pos] -= h
            fd = (o.lb_loss_from_logits(zp, k, routing, alpha)[0] - o.lb_loss_from_logits(zm, k, routing, alpha)[0]) / (2 * h)
            assert abs(fd - dz[pos]) < 1e-8
        np.testing.assert_allclose(dz.sum(axis=1), 0.0, atol=1e-15)
    # with u held constant only the p-term remains: gradient of alpha E sum_i u_i p_i(z) at fixed u
    k, routing = 2, o.ROUTE_TOPK
    dz = o.lb_loss_grad(z, k, routing, alpha, lb_stopgrad_u=True)
    _, u, _ = o.lb_loss_from_logits(z, k, routing, alpha)
    f = lambda zz: alpha * 4 * float(np.sum(u * o.full_softmax(zz).mean(axis=0)))
    pos = (3, 1)
    zp = z.copy(); zp[pos] += 1e-6
    zm = z.copy(); zm[pos] -= 1e-6
    assert abs((f(zp) - f(zm)) / 2e-6 - dz[pos]) < 1e-8


def test_router_gradient_rows_sum_to_zero():
    x, wr, w1, w3, w2, dy = small_problem(12)
    for routing, k in [(o.ROUTE_TOPK, 2), (o.ROUTE_SWITCH, 1), (o.ROUTE_SOFT, 4)]:
        g = o.moe_backward(x, wr, w1, w3, w2, dy, k=k, routing=routing, alpha=0.3)
        np.testing.assert_allclose(g["dlogits"].sum(axis=1), 0.0, atol=1e-13)
        np.testing.assert_allclose(g["dw_router"].sum(axis=0), 0.0, atol=1e-12)
        np.testing.assert_allclose(g["dbias"].sum(), 0.0, atol=1e-12)


def test_linearity_in_w2_and_gate_gradient_identity():
    x, wr, w1, w3, w2, dy = small_problem(13)
    a = o.moe_forward(x, wr, w1, w3, w2, k=2)
    b = o.moe_forward(x, wr, w1, w3, 2.5 * w2, k=2)
    np.testing.assert_allclose(b["y"], 2.5 * a["y"], rtol=1e-12, atol=1e-14)
    ga = o.moe_backward(x, wr, w1, w3, w2, dy, k=2, alpha=0.0)
    gb = o.moe_backward(x, wr, w1, w3, 2.5 * w2, dy, k=2, alpha=0.0)
    np.testing.assert_allclose(gb["dw1"], 2.5 * ga["dw1"], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(gb["dw2"], ga["dw2"], rtol=1e-11, atol=1e-13)
    # d/d gate = <dY_t, FF_i(x_t)> = <W2_i^T dY_t, a_{t,i}>
    idx = a["topk_idx"]
    for t in (0, 5, 17):
        for s in range(2):
            e = idx[t, s]
            _, _, _, act = o.swiglu_ffn(x[t:t + 1], w1[e], w3[e], w2[e], return_hidden=True)
            np.testing.assert_allclose(ga["dgate"][t, s], float((dy[t] @ w2[e]) @ act[0]), rtol=1e-11)


def test_slice_modes_agree_with_full_backward():
    x, wr, w1, w3, w2, dy = small_problem(14, T=30)
    for routing, k in [(o.ROUTE_TOPK, 2), (o.ROUTE_SWITCH, 1)]:
        full = o.moe_backward(x, wr, w1, w3, w2, dy, k=k, routing=routing, alpha=0.2, lb_grad_scale=0.9)
        fwd = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=0.2)
        tok = np.array([3, 4, 11, 29])
        sl = o.moe_backward_token_slice(x, wr, w1, w3, w2, dy, fwd["topk_idx"], fwd["gates"], fwd["probs"],
                                        fwd["u"], fwd["p"], tok, routing=routing, alpha=0.2, lb_grad_scale=0.9)
        np.testing.assert_allclose(sl["dx"], full["dx"][tok], rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(sl["dlogits"], full["dlogits"][tok], rtol=1e-11, atol=1e-14)
        ys = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, tokens=tok)["y"]
        np.testing.assert_allclose(ys, fwd["y"][tok], rtol=1e-12, atol=1e-14)
        J = np.array([0, 7, 19])
        for e in range(4):
            d1, d3, d2 = o.expert_wgrad_hidden_slice(x, w1, w3, w2, dy, fwd["topk_idx"], fwd["gates"], e, J)
            np.testing.assert_allclose(d1, full["dw1"][e][J], rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(d3, full["dw3"][e][J], rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(d2, full["dw2"][e][:, J], rtol=1e-11, atol=1e-13)


def test_router_gradient_from_a_supplied_dz():
    # closed form: dz nonzero at one (token, expert) entry only -> that row of dW_l is dz * x_t, dbias picks it up
    x, wr, w1, w3, w2, dy = small_problem(31, T=9, d=5)
    dz = np.zeros((9, 4))
    dz[6, 2] = -1.5
    dw, db = o.router_wgrad_from_dz(x, dz)
    want = np.zeros((4, 5))
    want[2] = -1.5 * x[6]
    np.testing.assert_allclose(dw, want, rtol=0, atol=1e-15)
    np.testing.assert_allclose(db, [0.0, 0.0, -1.5, 0.0], rtol=0, atol=0)
    # scalar loops on a tiny case (operand orientation: [E, d], not [d, E])
    r = RNG(32)
    dz = r.standard_normal((9, 4))
    dw, db = o.router_wgrad_from_dz(x, dz)
    for e in range(4):
        assert abs(db[e] - sum(dz[t, e] for t in range(9))) < 1e-13
        for c in range(5):
            assert abs(dw[e, c] - sum(dz[t, e] * x[t, c] for t in range(9))) < 1e-13
    # fed the full backward's own dz it reproduces that backward's router gradients (which finite differences pin)
    full = o.moe_backward(x, wr, w1, w3, w2, dy, k=2, alpha=0.3)
    dw, db = o.router_wgrad_from_dz(x, full["dlogits"])
    np.testing.assert_allclose(dw, full["dw_router"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(db, full["dbias"], rtol=1e-12, atol=1e-14)
    with pytest.raises(ValueError):
        o.router_wgrad_from_dz(x, dz[:5])


def test_logits_override_decides_routing():
    x, wr, w1, w3, w2, _ = small_problem(15)
    z32 = o.router_logits(x, wr).astype(np.float32)
    z32[0, :] = [1.0, 1.0, 1.0, 0.0]                      # a three-way tie decided by index
    out = o.moe_forward(x, wr, w1, w3, w2, k=2, logits=z32)
    assert out["topk_idx"][0].tolist() == [0, 1]
    np.testing.assert_allclose(out["gates"][0], [0.5, 0.5])


# ---- merge ------------------------------------------------------------------------------------

def test_merge_pins():
    r = RNG(16)
    seed_model = {"layers.0.attn.wq": r.standard_normal((8, 8)).astype(np.float32),
                  "layers.0.ffn.w1": r.standard_normal((5, 8)).astype(np.float32),
                  "norm": r.standard_normal(8).astype(np.float32)}
    for n in (2, 4):                                      # power of two: exact
        m = o.merge_models([seed_model] * n, "f32")
        assert (m["layers.0.attn.wq"] == seed_model["layers.0.attn.wq"]).all()
        assert (m["norm"] == seed_model["norm"]).all()
        assert m["layers.0.ffn.w1"].shape == (n, 5, 8)
        for e in range(n):
            assert (m["layers.0.ffn.w1"][e] == seed_model["layers.0.ffn.w1"]).all()
    m3 = o.merge_models([seed_model] * 3, "f32")          # (3 a)/3 may differ by an ulp
    np.testing.assert_allclose(m3["norm"], seed_model["norm"], rtol=2e-7)
    a = {"norm": np.array([1.0, 2.0, -4.0])}
    b = {"norm": np.array([3.0, 2.5, 4.0])}
    assert o.merge_models([a, b], "f32")["norm"].tolist() == [2.0, 2.25, 0.0]
    # experts keep their order
    ma = {"l.ffn.w2": np.full((2, 2), 1.0)}; mb = {"l.ffn.w2": np.full((2, 2), 2.0)}
    st = o.merge_models([ma, mb], "f32")["l.ffn.w2"]
    assert (st[0] == 1.0).all() and (st[1] == 2.0).all()


def test_bf16_rounding_against_torch_and_ties():
    # ties to even at 8 significant bits
    v = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -9, -(1.0 + 2.0 ** -8), 0.0, 3.0e-40])
    got = o.round_to_bf16(v)
    assert got[:5].tolist() == [1.0, 1.0 + 2.0 ** -6, 1.0, -1.0, 0.0]
    # fp32 inputs: torch's own float32 -> bfloat16 conversion is an independent implementation
    r = RNG(17)
    f = (r.standard_normal(20000) * np.exp(r.uniform(-20, 20, 20000))).astype(np.float32)
    want = torch.from_numpy(f).to(torch.bfloat16).to(torch.float64).numpy()
    assert (o.round_to_bf16(f.astype(np.float64)) == want).all()
    # mean of bf16 values rounded once
    a = torch.from_numpy(f[:1000]).to(torch.bfloat16)
    b = torch.from_numpy(f[1000:2000]).to(torch.bfloat16)
    m = o.merge_average([a.to(torch.float64).numpy(), b.to(torch.float64).numpy()], "bf16")
    want = ((a.to(torch.float32) + b.to(torch.float32)) / 2).to(torch.bfloat16).to(torch.float64).numpy()
    # a + b of two bf16 numbers is exact in fp32 unless their exponents differ by more than 16
    close = np.abs(np.log2(np.abs(a.float().numpy()) / np.abs(b.float().numpy()))) < 14
    assert (m[close] == want[close]).all()


def test_table4_active_parameter_counts():
    path = os.path.join(os.path.dirname(__file__), "golden", "table4_active_params.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for name, k, printed in rows:
        n = o.active_parameters(32, 4096, 11008, 32000, 4, int(k))
        assert round(n / 1e9, 1) == float(printed), (name, n)
    # the same table fixes the split used by the merge workload
    shapes = o.llama_like_param_shapes(32, 4096, 11008, 32000)
    ffn = sum(int(np.prod(s)) for n, s in shapes if ".ffn." in n)
    other = sum(int(np.prod(s)) for n, s in shapes if ".ffn." not in n)
    assert ffn == 4_328_521_728 and other == 2_409_893_888


# ---- Sample Top-1 routing (Gumbel softmax, keep the largest entry) ----------------------------

def test_sample_top1_reduces_to_switch_without_noise():
    x, wr, w1, w3, w2, dy = small_problem(21, scale_r=1.5)
    zero = np.zeros((x.shape[0], 4))
    a = o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SWITCH, alpha=0.0)
    b = o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=zero, tau=1.0)
    assert (a["topk_idx"] == b["topk_idx"]).all()
    np.testing.assert_allclose(a["y"], b["y"], rtol=1e-13)
    ga = o.moe_backward(x, wr, w1, w3, w2, dy, k=1, routing=o.ROUTE_SWITCH, alpha=0.0)
    gb = o.moe_backward(x, wr, w1, w3, w2, dy, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=zero, tau=1.0)
    np.testing.assert_allclose(ga["dw_router"], gb["dw_router"], rtol=1e-12, atol=1e-14)


def test_sample_top1_selection_and_temperature_limits():
    r = RNG(22)
    x, wr, w1, w3, w2, _ = small_problem(22)
    noise = -np.log(-np.log(r.uniform(size=(x.shape[0], 4))))
    z = o.router_logits(x, wr)
    out = o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=0.7)
    assert (out["topk_idx"][:, 0] == np.argmax(z + noise, axis=1)).all()
    soft = np.exp((z + noise) / 0.7); soft /= soft.sum(1, keepdims=True)
    np.testing.assert_allclose(out["gates"][:, 0], soft.max(axis=1), rtol=1e-13)   # the kept entry of the soft sample
    np.testing.assert_allclose(out["logits"], z, rtol=1e-14)                        # reported logits are unperturbed
    sharp = o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=1e-3)
    np.testing.assert_allclose(sharp["gates"], 1.0, atol=1e-6)                      # annealed: a sharp distribution
    hard = o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=0.0)
    assert (hard["gates"] == 1.0).all() and (hard["topk_idx"] == out["topk_idx"]).all()
    e = hard["topk_idx"][:, 0]
    want = np.stack([o.swiglu_ffn(x[t:t + 1], w1[e[t]], w3[e[t]], w2[e[t]])[0] for t in range(x.shape[0])])
    np.testing.assert_allclose(hard["y"], want, rtol=1e-12, atol=1e-13)


def test_sample_top1_selection_in_fp32_ties_like_an_fp32_implementation():
    # z + G differs between the experts only below fp32 resolution: 1 + 2^-25 rounds to 1 in fp32.
    # In fp64 expert 1 wins; an fp32 implementation sees a tie, which goes to the lower index.
    z = np.array([[0.0, 2.0 ** -25, -3.0]], dtype=np.float32)
    G = np.array([[1.0, 1.0, 0.0]], dtype=np.float32)
    for tau in (0.0, 0.8):
        _, idx64, _, _ = o.route(None, None, 1, o.ROUTE_SAMPLE1, logits=z, noise=G, tau=tau)
        _, idx32, g32, p32 = o.route(None, None, 1, o.ROUTE_SAMPLE1, logits=z, noise=G, tau=tau, select_fp32=True)
        assert idx64.tolist() == [[1]] and idx32.tolist() == [[0]]
        # the gate is still the fp64 softmax entry of the chosen expert (1 for hard sampling)
        want = 1.0 if tau == 0.0 else float(o.full_softmax((z.astype(np.float64) + G) / tau)[0, 0])
        assert abs(float(g32[0, 0]) - want) < 1e-15
    # where fp32 resolves the two sums the flag changes nothing
    z2 = np.array([[0.0, 2.0 ** -20, -3.0]], dtype=np.float32)
    _, a, _, _ = o.route(None, None, 1, o.ROUTE_SAMPLE1, logits=z2, noise=G, tau=0.5)
    _, b, _, _ = o.route(None, None, 1, o.ROUTE_SAMPLE1, logits=z2, noise=G, tau=0.5, select_fp32=True)
    assert a.tolist() == b.tolist() == [[1]]


def test_hard_sampling_follows_the_softmax_distribution():
    # Gumbel-max: arg-max(z + G) is a draw from SoftMax(z)
    r = RNG(23)
    z = np.tile(np.array([[1.0, 0.0, -0.5, 2.0]]), (40000, 1))
    noise = -np.log(-np.log(r.uniform(size=z.shape)))
    _, idx, _, _ = o.route(None, None, 1, o.ROUTE_SAMPLE1, logits=z, noise=noise, tau=0.0)
    freq = np.bincount(idx[:, 0], minlength=4) / z.shape[0]
    np.testing.assert_allclose(freq, o.full_softmax(z[:1])[0], atol=0.01)


def test_sample_top1_gradients_against_finite_differences():
    x, wr, w1, w3, w2, G = small_problem(24, T=10, d=6, F=7, E=4, scale_r=1.5)
    r = RNG(25)
    noise = -np.log(-np.log(r.uniform(size=(10, 4))))
    tau = 0.8
    zs = np.sort(o.router_logits(x, wr) + noise, axis=1)
    assert np.min(np.diff(zs, axis=1)) > 1e-3
    g = o.moe_backward(x, wr, w1, w3, w2, G, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=tau)
    f = lambda: float(np.sum(o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0,
                                           noise=noise, tau=tau)["y"] * G))
    h = 1e-6
    for arr, name in ((x, "dx"), (wr, "dw_router"), (w2, "dw2"), (w1, "dw1")):
        for _ in range(6):
            pos = tuple(int(r.integers(0, s)) for s in arr.shape)
            old = arr[pos]
            arr[pos] = old + h; lp = f()
            arr[pos] = old - h; lm = f()
            arr[pos] = old
            fd = (lp - lm) / (2 * h)
            assert abs(fd - g[name][pos]) <= 2e-6 * max(1.0, abs(fd)), (name, pos, fd, g[name][pos])
    hard = o.moe_backward(x, wr, w1, w3, w2, G, k=1, routing=o.ROUTE_SAMPLE1, alpha=0.0, noise=noise, tau=0.0)
    assert np.all(hard["dw_router"] == 0.0)


# ---- split / blend layouts of the merge ---------------------------------------------------------

def test_split_and_blend_layouts_preserve_the_feed_forward_sums():
    r = RNG(31)
    N, F, d = 4, 24, 6
    w1s = [r.standard_normal((F, d)) for _ in range(N)]
    w3s = [r.standard_normal((F, d)) for _ in range(N)]
    w2s = [r.standard_normal((d, F)) for _ in range(N)]
    x = r.standard_normal((5, d))
    ff = [o.swiglu_ffn(x, w1s[i], w3s[i], w2s[i]) for i in range(N)]
    # splitting: the un-gated sum of the chunks of model i is FF_i (SwiGLU acts per hidden unit)
    for C in (1, 2, 3):
        s1, s3, s2 = o.merge_ffn_layout(w1s, w3s, w2s, o.FFN_SPLIT, C)
        assert s1.shape == (N * C, F // C, d) and s2.shape == (N * C, d, F // C)
        for i in range(N):
            tot = sum(o.swiglu_ffn(x, s1[i * C + c], s3[i * C + c], s2[i * C + c]) for c in range(C))
            np.testing.assert_allclose(tot, ff[i], rtol=1e-12, atol=1e-13)
    # blending: every expert has the full width and the sum over all experts is the sum over all models
    b1, b3, b2 = o.merge_ffn_layout(w1s, w3s, w2s, o.FFN_BLEND)
    assert b1.shape == (N, F, d) and b2.shape == (N, d, F)
    np.testing.assert_allclose(sum(o.swiglu_ffn(x, b1[n], b3[n], b2[n]) for n in range(N)), sum(ff), rtol=1e-12, atol=1e-13)
    # expert n of the blend starts with the n-th chunk of model 0
    Fc = F // N
    assert (b1[2][:Fc] == w1s[0][2 * Fc:3 * Fc]).all() and (b2[2][:, Fc:2 * Fc] == w2s[1][:, 2 * Fc:3 * Fc]).all()
    # blending identical models permutes hidden units only: each expert equals the seed FF
    same = o.merge_ffn_layout([w1s[0]] * N, [w3s[0]] * N, [w2s[0]] * N, o.FFN_BLEND)
    for n in range(N):
        got = o.swiglu_ffn(x, same[0][n], same[1][n], same[2][n])
        want = N * o.swiglu_ffn(x, w1s[0][n * Fc:(n + 1) * Fc], w3s[0][n * Fc:(n + 1) * Fc], w2s[0][:, n * Fc:(n + 1) * Fc])
        np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-13)
    st = o.merge_ffn_layout(w1s, w3s, w2s, o.FFN_STACK)
    assert (st[0][1] == w1s[1]).all() and (st[2][3] == w2s[3]).all()


# ---- capacity factor (Section 4.1: Switch routing with a hard limit, beyond which tokens drop) ---

def test_capacity_closed_forms_and_worked_example():
    assert o.expert_capacity(16384, 1, 4, 1.5) == 6144           # the paper's CF on the bench batch
    assert o.expert_capacity(10, 1, 4, 1.0) == 3                 # ceil(2.5)
    assert o.expert_capacity(10, 2, 4, 1.0) == 5
    assert o.expert_capacity(7, 1, 4, 0.0) == 7                  # 0 = no limit
    idx = np.array([[0], [0], [1], [0], [1], [0], [2]])
    keep = o.capacity_keep(idx, 3, 2)
    assert keep[:, 0].tolist() == [True, True, True, False, True, False, True]
    counts, offsets, perm, inv_perm = o.dispatch(idx, 3, keep)
    assert counts.tolist() == [2, 2, 1] and offsets.tolist() == [0, 2, 4, 5]
    assert perm.tolist() == [0, 1, 2, 4, 6, -1, -1]
    assert inv_perm.tolist() == [0, 1, 2, -1, 3, -1, 4]
    # top-2: slots of one token are taken in slot order
    idx2 = np.array([[0, 1], [1, 0], [0, 1]])
    assert o.capacity_keep(idx2, 2, 2).tolist() == [[True, True], [True, True], [False, False]]


def test_capacity_forward_drops_exactly_the_overflow():
    x, wr, w1, w3, w2, dy = small_problem(31, T=40, scale_r=2.0)
    for routing, k in [(o.ROUTE_SWITCH, 1), (o.ROUTE_TOPK, 2)]:
        free = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=0.3)
        # a limit nobody reaches changes nothing
        big = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=0.3, capacity_factor=4.0)
        assert np.array_equal(big["y"], free["y"]) and np.array_equal(big["perm"], free["perm"])
        cf = 0.6
        cap = o.expert_capacity(40, k, 4, cf)
        assert max(free["counts"]) > cap                          # the case does drop
        lim = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=0.3, capacity_factor=cf)
        assert lim["counts"].tolist() == [min(int(c), cap) for c in free["counts"]]
        # router outputs and the loss are those of the router, whatever is dropped
        for name in ("topk_idx", "gates", "probs", "u", "p"):
            assert np.array_equal(lim[name], free[name])
        assert lim["lb_loss"] == free["lb_loss"]
        # y of a token: the sum over its kept slots only, each term as without a limit
        for t in range(40):
            want = np.zeros(12)
            for slot in range(k):
                if lim["keep"][t, slot]:
                    e = int(free["topk_idx"][t, slot])
                    want += free["gates"][t, slot] * o.swiglu_ffn(x[t:t + 1], w1[e], w3[e], w2[e])[0]
            np.testing.assert_allclose(lim["y"][t], want, rtol=1e-12, atol=1e-14)
        # per expert the kept ones are the first `cap` in token order
        for e in range(4):
            flat = [t * k + s for t in range(40) for s in range(k) if free["topk_idx"][t, s] == e]
            kept = [f for f in flat if lim["keep"][f // k, f % k]]
            assert kept == flat[:cap]
            assert lim["perm"][lim["offsets"][e]:lim["offsets"][e + 1]].tolist() == kept


def test_capacity_backward_equals_backward_on_the_kept_sub_batch():
    """Switch routing, alpha = 0: the step with a limit is the step without one on the kept tokens
    (same logits), and a dropped token receives no gradient at all."""
    x, wr, w1, w3, w2, dy = small_problem(32, T=36, scale_r=2.0)
    cf = 0.5
    fwd = o.moe_forward(x, wr, w1, w3, w2, k=1, routing=o.ROUTE_SWITCH, alpha=0.0, capacity_factor=cf)
    keep = fwd["keep"][:, 0]
    assert 0 < keep.sum() < 36
    g = o.moe_backward(x, wr, w1, w3, w2, dy, k=1, routing=o.ROUTE_SWITCH, alpha=0.0, capacity_factor=cf)
    sub = o.moe_backward(x[keep], wr, w1, w3, w2, dy[keep], k=1, routing=o.ROUTE_SWITCH, alpha=0.0)
    for name in ("dw1", "dw3", "dw2", "dw_router", "dbias"):
        np.testing.assert_allclose(g[name], sub[name], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(g["dx"][keep], sub["dx"], rtol=1e-11, atol=1e-13)
    assert np.all(g["dx"][~keep] == 0.0) and np.all(g["dlogits"][~keep] == 0.0)


def test_capacity_gradients_against_finite_differences_and_slices():
    x, wr, w1, w3, w2, G = small_problem(33, T=14, d=6, F=7, E=4, scale_r=1.5)
    alpha, lam, cf = 0.7, 1.3, 0.6
    z = o.router_logits(x, wr)
    assert np.min(np.diff(np.sort(z, axis=1), axis=1)) > 1e-3
    for routing, k in [(o.ROUTE_SWITCH, 1), (o.ROUTE_TOPK, 2)]:
        fwd = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=alpha, capacity_factor=cf)
        assert not fwd["keep"].all()
        g = o.moe_backward(x, wr, w1, w3, w2, G, k=k, routing=routing, alpha=alpha, lb_grad_scale=lam,
                           capacity_factor=cf)

        def loss():
            out = o.moe_forward(x, wr, w1, w3, w2, k=k, routing=routing, alpha=alpha, capacity_factor=cf)
            return float(np.sum(out["y"] * G)) + lam * out["lb_loss"]

        r = RNG(5)
        h = 1e-6
        for pname, arr, gname in [("x", x, "dx"), ("wr", wr, "dw_router"), ("w1", w1, "dw1"), ("w3", w3, "dw3"),
                                  ("w2", w2, "dw2")]:
            for _ in range(8):
                pos = tuple(int(r.integers(0, s)) for s in arr.shape)
                old = arr[pos]
                arr[pos] = old + h
                lp = loss()
                arr[pos] = old - h
                lm = loss()
                arr[pos] = old
                fd = (lp - lm) / (2 * h)
                assert abs(fd - g[gname][pos]) <= 2e-6 * max(1.0, abs(fd)), (pname, pos, fd, g[gname][pos])
        # the slice forms agree with the full backward under a limit
        tok = np.arange(14)
        sl = o.moe_backward_token_slice(x, wr, w1, w3, w2, G, fwd["topk_idx"], fwd["gates"], fwd["probs"],
                                        fwd["u"], fwd["p"], tok, routing=routing, alpha=alpha, lb_grad_scale=lam,
                                        keep=fwd["keep"])
        np.testing.assert_allclose(sl["dx"], g["dx"], rtol=1e-11, atol=1e-13)
        J = np.array([1, 6])
        for e in range(4):
            d1, d3, d2 = o.expert_wgrad_hidden_slice(x, w1, w3, w2, G, fwd["topk_idx"], fwd["gates"], e, J,
                                                     keep=fwd["keep"])
            np.testing.assert_allclose(d1, g["dw1"][e][J], rtol=1e-11, atol=1e-13)
            np.testing.assert_allclose(d2, g["dw2"][e][:, J], rtol=1e-11, atol=1e-13)
