"""Plain CPU oracle (float64, numpy) for the Branch-Train-MiX MoE feed-forward sublayer.

TEST INFRASTRUCTURE ONLY.  This module exists so that tests, the smoke check and the
timed CPU baseline have a slow, obviously-correct statement of what the layer computes.
Nothing on the product path may import it, and it imports nothing from the CUDA package.

Every function is the definition written out with numpy in float64: no tiling, no fusion,
no re-association beyond what the cited formula states.  Inputs that were stored as
bf16/fp32 convert to float64 exactly, so the only rounding is float64's own.

What each part follows (paper = arXiv 2403.07816):
  * router logits, top-k routing, gate softmax ......... Section 3.2, the FF_MoE equation and
                                                          g(W_l x) = SoftMax(TopK(W_l x))
  * expert feed-forward FF_i ........................... Section 3.2 ("feedforward sublayer" of a
                                                          Llama-2 seed, Section 4.1): SwiGLU
                                                          W2 (silu(W1 x) * W3 x), no biases
  * load-balancing loss ................................ Section 3.3, the L_LB equation
  * Switch / soft / Sample Top-1 routing ............... Section 3.3, "Routing method"
  * merge (stack FFNs, average the rest) ............... Section 3.2, the two paragraphs after
                                                          the routing formula
  * backward ........................................... derivatives of the above (MoE finetuning,
                                                          Sections 1 and 3.2), checked by finite
                                                          differences in the tests

Readings where the paper is silent (each is also listed in the design notes):
  * top-k ties go to the lower expert index; slot 0 holds the largest logit;
  * Switch routing uses the full-softmax probability of the arg-max expert as its gate;
  * u_i in L_LB is the batch mean of the gate VALUE, exactly as printed, and the loss is
    differentiated through both u and p unless `lb_stopgrad_u` is set;
  * N in "alpha N" is the number of experts in the layer; the batch is all T tokens of a call;
  * the merge average is uniform over all N models, one rounding to the storage type at the end.

Parity status: every function here is pinned by tests/test_oracle_pins.py (closed forms,
invariants, brute force, finite differences, the paper's Table 4 parameter counts).
"""
from __future__ import annotations

import math

import numpy as np

ROUTE_TOPK = 0
ROUTE_SWITCH = 1
ROUTE_SOFT = 2
ROUTE_SAMPLE1 = 3

_F64 = np.float64


def _f64(a):
    return np.asarray(a, dtype=_F64)


# --------------------------------------------------------------------------------------
# Router (Section 3.2: logits = W_l x; g = SoftMax(TopK(.)))
# --------------------------------------------------------------------------------------

def router_logits(x, w_router, router_bias=None):
    """z[t, i] = sum_c W_l[i, c] * x[t, c]  (+ b_i; the bias is not in the paper)."""
    z = _f64(x) @ _f64(w_router).T
    if router_bias is not None:
        z = z + _f64(router_bias)[None, :]
    return z


def top_k_select(z, k):
    """Indices of the k largest logits per token, slot 0 = largest.

    Selection is by repeated arg-max; numpy's argmax returns the first occurrence of the
    maximum, which is the lower expert index on a tie (and -0.0 == +0.0 compares equal).
    """
    z = np.asarray(z)
    T, E = z.shape
    if not (1 <= k <= E):
        raise ValueError("need 1 <= k <= E")
    if not np.all(np.isfinite(z)):
        raise ValueError("logits must be finite")
    work = z.astype(_F64).copy()
    idx = np.empty((T, k), dtype=np.int32)
    rows = np.arange(T)
    for j in range(k):
        best = np.argmax(work, axis=1)
        idx[:, j] = best
        work[rows, best] = -np.inf
    return idx


def full_softmax(z):
    """SoftMax_i(W_l x) over all experts (the p of Section 3.3)."""
    z = _f64(z)
    m = z.max(axis=1, keepdims=True)
    e = np.exp(z - m)
    return e / e.sum(axis=1, keepdims=True)


def gate_values(z, idx, routing=ROUTE_TOPK):
    """Gate weight of each selected expert, shape [T, k].

    TOPK / SOFT: softmax restricted to the selected logits (Section 3.2).
    SWITCH: probability of the arg-max under the full softmax (Section 3.3).
    """
    z = _f64(z)
    T = z.shape[0]
    sel = np.take_along_axis(z, idx.astype(np.int64), axis=1)
    if routing == ROUTE_SWITCH:
        if idx.shape[1] != 1:
            raise ValueError("Switch routing selects exactly one expert")
        return np.take_along_axis(full_softmax(z), idx.astype(np.int64), axis=1)
    m = sel.max(axis=1, keepdims=True)
    e = np.exp(sel - m)
    return e / e.sum(axis=1, keepdims=True)


def dense_gates(idx, gates, E):
    """g_i(W_l x) as a [T, E] array with zeros for the experts that were not selected."""
    T, k = idx.shape
    g = np.zeros((T, E), dtype=_F64)
    g[np.arange(T)[:, None], idx.astype(np.int64)] = _f64(gates)
    return g


# --------------------------------------------------------------------------------------
# Load-balancing loss (Section 3.3)
# --------------------------------------------------------------------------------------

def lb_loss(gates_dense, probs, alpha):
    """L_LB = alpha * N * sum_i u_i p_i, u_i = batch mean of g_i, p_i = batch mean of SoftMax_i."""
    g = _f64(gates_dense)
    p_tok = _f64(probs)
    E = g.shape[1]
    u = g.mean(axis=0)
    p = p_tok.mean(axis=0)
    return float(alpha) * E * float(np.sum(u * p)), u, p


def lb_loss_from_logits(z, k, routing, alpha):
    """The whole Section 3.3 loss from logits: (loss, u, p)."""
    E = np.asarray(z).shape[1]
    kk = E if routing == ROUTE_SOFT else k
    idx = top_k_select(z, kk)
    g = gate_values(z, idx, routing)
    return lb_loss(dense_gates(idx, g, E), full_softmax(z), alpha)


# --------------------------------------------------------------------------------------
# Dispatch permutation (implementation structure: assignments sorted by expert, then token)
# --------------------------------------------------------------------------------------

def expert_capacity(T, k, E, capacity_factor):
    """Rows one expert accepts: ceil(CF * T * k / E), CF held as an fp32 number (Section 4.1 sets
    CF = 1.5 for Switch routing, where k = 1; 0 means no limit)."""
    cf = float(np.float32(capacity_factor))
    if cf <= 0.0:
        return T * k
    return int(math.ceil(cf * float(T * k) / float(E)))


def capacity_keep(idx, E, capacity):
    """keep[T, k]: an expert takes its assignments in order of flat id (token, then slot) until it
    holds `capacity` of them; the hard limit of Section 4.1 drops the rest."""
    idx = np.asarray(idx)
    T, k = idx.shape
    keep = np.zeros((T, k), dtype=bool)
    held = [0] * E
    for t in range(T):
        for slot in range(k):
            e = int(idx[t, slot])
            if held[e] < capacity:
                held[e] += 1
                keep[t, slot] = True
    return keep


def dispatch(idx, E, keep=None):
    """counts[E], offsets[E+1], perm[R], inv_perm[R] for the R = T*k assignments.

    Assignment (t, slot) has flat id t*k + slot.  Sorted order is by expert id ascending and,
    inside one expert, by token index ascending (a token meets an expert at most once).
    perm[r] = flat id of the assignment in sorted row r; inv_perm[flat id] = r.
    With `keep` (capacity limit) only kept assignments are counted and sorted: a dropped one has
    inv_perm = -1 and the unused tail of perm is -1.
    """
    idx = np.asarray(idx)
    T, k = idx.shape
    flat = idx.reshape(-1).astype(np.int64)
    kept = np.ones(T * k, dtype=bool) if keep is None else np.asarray(keep, dtype=bool).reshape(-1)
    counts = np.zeros(E, dtype=np.int32)
    for e in range(E):
        counts[e] = int(np.sum((flat == e) & kept))
    offsets = np.zeros(E + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(counts)
    order = np.argsort(flat, kind="stable")
    order = order[kept[order]]
    perm = np.full(T * k, -1, dtype=np.int32)
    perm[:len(order)] = order
    inv_perm = np.full(T * k, -1, dtype=np.int32)
    inv_perm[order] = np.arange(len(order), dtype=np.int32)
    return counts, offsets, perm, inv_perm


# --------------------------------------------------------------------------------------
# Expert feed-forward (SwiGLU)
# --------------------------------------------------------------------------------------

def sigmoid(v):
    return 1.0 / (1.0 + np.exp(-v))


def swiglu_ffn(x, w1, w3, w2, return_hidden=False):
    """FF(x) = W2 (silu(W1 x) * (W3 x)) for row-vector tokens x[T, d]; W1, W3: [F, d], W2: [d, F]."""
    x = _f64(x)
    h1 = x @ _f64(w1).T
    h3 = x @ _f64(w3).T
    a = h1 * sigmoid(h1) * h3
    y = a @ _f64(w2).T
    if return_hidden:
        return y, h1, h3, a
    return y


# --------------------------------------------------------------------------------------
# MoE forward
# --------------------------------------------------------------------------------------

def route(x, w_router, k, routing=ROUTE_TOPK, router_bias=None, logits=None, noise=None, tau=1.0,
          select_fp32=False):
    """Steps 1-4: logits (or the caller's fp32 logits), selection, gates, full softmax.

    ROUTE_SAMPLE1 (Section 3.3, "Sample Top-1"): with Gumbel noise G (an input) the soft sample is
    SoftMax((z + G) / tau); only its largest entry is kept as the gate of that one expert.  tau = 0
    is the inference rule, hard sampling: the expert arg-max(z + G) with gate 1.  For this mode the
    returned probabilities are those of the perturbed logits (the quantity the gate is taken from).

    `select_fp32`: the arg-max of Sample Top-1 is an integer decided by floating point.  When the
    routing of an fp32 implementation is to be reproduced bit for bit (its fp32 logits and the fp32
    noise are passed in), the perturbed logits that DECIDE the expert are formed the way that
    implementation forms them, by one fp32 addition z + G, so that two sums that fp32 rounds to the
    same number tie here as well (and go to the lower index).  Gate and probabilities stay fp64.
    """
    z = router_logits(x, w_router, router_bias) if logits is None else _f64(logits)
    E = z.shape[1]
    kk = E if routing == ROUTE_SOFT else k
    if routing in (ROUTE_SWITCH, ROUTE_SAMPLE1) and kk != 1:
        raise ValueError("Switch and Sample Top-1 routing need k = 1")
    if routing == ROUTE_SAMPLE1:
        if noise is None:
            raise ValueError("Sample Top-1 routing needs the Gumbel noise")
        zp = z + _f64(noise)
        if select_fp32:
            idx = top_k_select(np.asarray(z, dtype=np.float32) + np.asarray(noise, dtype=np.float32), 1)
        else:
            idx = top_k_select(zp, 1)
        if tau > 0:
            zp = zp / float(tau)
            p = full_softmax(zp)
            g = np.take_along_axis(p, idx.astype(np.int64), axis=1)
        else:
            p = full_softmax(zp)
            g = np.ones((z.shape[0], 1), dtype=_F64)
        return z, idx, g, p
    idx = top_k_select(z, kk)
    g = gate_values(z, idx, routing)
    p = full_softmax(z)
    return z, idx, g, p


def moe_forward(x, w_router, w1, w3, w2, k, routing=ROUTE_TOPK, alpha=0.01,
                router_bias=None, logits=None, tokens=None, noise=None, tau=1.0, capacity_factor=0.0,
                select_fp32=False):
    """FF_MoE(x) = sum_i g_i(W_l x) FF_i(x), skipping experts whose gate is zero.

    capacity_factor > 0 (Section 4.1, Switch routing): an assignment beyond its expert's capacity
    is dropped, i.e. contributes nothing to y; gates, probabilities and L_LB are those of the router.

    w1, w3: [E, F, d]; w2: [E, d, F].  `logits` (optional, [T, E]) replaces W_l x so that the
    routing decision can be taken on exactly the numbers another implementation produced.
    `tokens` (optional index array) restricts the expert computation to those tokens; routing
    and the loss always use every token.  Returns a dict.
    """
    x = _f64(x)
    T, d = x.shape
    E = np.asarray(w1).shape[0]
    z, idx, g, p_tok = route(x, w_router, k, routing, router_bias, logits, noise, tau, select_fp32)
    gd = dense_gates(idx, g, E)
    loss, u, p = lb_loss(gd, p_tok, alpha)
    kk = idx.shape[1]
    if capacity_factor > 0 and routing == ROUTE_SOFT:
        raise ValueError("a capacity limit has no meaning when every expert takes every token")
    keep = capacity_keep(idx, E, expert_capacity(T, kk, E, capacity_factor)) if capacity_factor > 0 \
        else np.ones(idx.shape, dtype=bool)
    counts, offsets, perm, inv_perm = dispatch(idx, E, keep)

    tok = np.arange(T) if tokens is None else np.asarray(tokens, dtype=np.int64)
    y = np.zeros((len(tok), d), dtype=_F64)
    for slot in range(kk):                       # slot order, as the combine is defined
        for e in range(E):
            m = (idx[tok, slot] == e) & keep[tok, slot]
            if not np.any(m):
                continue
            y[m] += g[tok[m], slot][:, None] * swiglu_ffn(x[tok[m]], w1[e], w3[e], w2[e])
    return dict(logits=z, topk_idx=idx, gates=g, probs=p_tok, y=y, lb_loss=loss, u=u, p=p,
                counts=counts, offsets=offsets, perm=perm, inv_perm=inv_perm, tokens=tok, keep=keep)


def moe_forward_all_experts(x, w_router, w1, w3, w2, k, routing=ROUTE_TOPK, router_bias=None):
    """The FF_MoE equation taken literally: every expert on every token, times its gate."""
    x = _f64(x)
    E = np.asarray(w1).shape[0]
    z, idx, g, _ = route(x, w_router, k, routing, router_bias)
    gd = dense_gates(idx, g, E)
    y = np.zeros_like(x)
    for i in range(E):
        y += gd[:, i:i + 1] * swiglu_ffn(x, w1[i], w3[i], w2[i])
    return y


# --------------------------------------------------------------------------------------
# MoE backward
# --------------------------------------------------------------------------------------

def router_backward_dz(idx, gates, probs, dgate, u, alpha, lb_grad_scale, routing=ROUTE_TOPK,
                       batch_size=None):
    """d(total loss)/d(logits) given d/d(gate value) of every selected expert.

    `dgate` already contains every path into the gate values (the main loss and, unless
    stopped, the u-term of L_LB).  This adds the softmax Jacobians and the p-term of L_LB.
    `batch_size` is |B| of the loss when the rows passed in are only part of the batch.
    """
    idx = np.asarray(idx).astype(np.int64)
    g = _f64(gates)
    p = _f64(probs)
    dg = _f64(dgate)
    T, E = p.shape
    B = T if batch_size is None else int(batch_size)
    rows = np.arange(T)[:, None]
    dz = np.zeros((T, E), dtype=_F64)
    if routing == ROUTE_SWITCH:
        # gate = p[argmax]; d gate / d z_j = p_sel (delta_j,sel - p_j)
        psel = np.take_along_axis(p, idx, axis=1)            # [T,1]
        dz += dg * psel * (-p)
        dz[rows, idx] += dg * psel
    else:
        inner = np.sum(g * dg, axis=1, keepdims=True)
        dz[rows, idx] += g * (dg - inner)
    # L_LB through p: d L_LB / d p_tok[t,i] = alpha E u_i / T
    c = lb_grad_scale * alpha * E * _f64(u) / B
    dz += p * (c[None, :] - (p @ c)[:, None])
    return dz


def moe_backward(x, w_router, w1, w3, w2, dy, k, routing=ROUTE_TOPK, alpha=0.01,
                 lb_grad_scale=1.0, lb_stopgrad_u=False, router_bias=None, logits=None, noise=None, tau=1.0,
                 capacity_factor=0.0, select_fp32=False):
    """Gradients of  <Y, dY> + lb_grad_scale * L_LB  w.r.t. x, W_l, bias, W1, W3, W2 (all tokens).
    A dropped assignment (capacity_factor > 0) is absent from Y, so nothing flows through it; the
    keep/drop decision itself is piecewise constant."""
    x = _f64(x)
    dy = _f64(dy)
    T, d = x.shape
    E, F, _ = np.asarray(w1).shape
    z, idx, g, p_tok = route(x, w_router, k, routing, router_bias, logits, noise, tau, select_fp32)
    if routing == ROUTE_SAMPLE1 and alpha != 0:
        raise ValueError("Sample Top-1 routing is defined here without the load-balancing loss (alpha = 0)")
    kk = idx.shape[1]
    gd = dense_gates(idx, g, E)
    _, u, p = lb_loss(gd, p_tok, alpha)
    keep = capacity_keep(idx, E, expert_capacity(T, kk, E, capacity_factor)) if capacity_factor > 0 \
        else np.ones(idx.shape, dtype=bool)

    dx = np.zeros_like(x)
    dw1 = np.zeros((E, F, d), dtype=_F64)
    dw3 = np.zeros((E, F, d), dtype=_F64)
    dw2 = np.zeros((E, d, F), dtype=_F64)
    dgate = np.zeros((T, kk), dtype=_F64)
    for slot in range(kk):
        for e in range(E):
            m = (idx[:, slot] == e) & keep[:, slot]
            if not np.any(m):
                continue
            xe = x[m]
            w1e, w3e, w2e = _f64(w1[e]), _f64(w3[e]), _f64(w2[e])
            y_e, h1, h3, a = swiglu_ffn(xe, w1e, w3e, w2e, return_hidden=True)
            dye = dy[m]
            dgate[m, slot] = np.sum(dye * y_e, axis=1)           # d/dg of g * y_e
            dout = g[m, slot][:, None] * dye                      # gradient reaching FF_e's output
            da = dout @ w2e
            dw2[e] += dout.T @ a
            s = sigmoid(h1)
            dh1 = da * h3 * s * (1.0 + h1 * (1.0 - s))
            dh3 = da * h1 * s
            dw1[e] += dh1.T @ xe
            dw3[e] += dh3.T @ xe
            dx[m] += dh1 @ w1e + dh3 @ w3e
    if not lb_stopgrad_u:
        # L_LB through u: d L_LB / d g[t,i] = alpha E p_i / T
        dgate += lb_grad_scale * alpha * E / T * p[idx.astype(np.int64)]
    if routing == ROUTE_SAMPLE1:
        # gate = SoftMax((z+G)/tau)[arg-max]: the Switch Jacobian in the perturbed logits, times 1/tau;
        # hard sampling (tau = 0) has a constant gate, hence no router gradient
        dz = (router_backward_dz(idx, g, p_tok, dgate, u, 0.0, 0.0, ROUTE_SWITCH) / float(tau)) if tau > 0 \
            else np.zeros((T, E), dtype=_F64)
    else:
        dz = router_backward_dz(idx, g, p_tok, dgate, u, alpha, lb_grad_scale, routing)
    dw_router = dz.T @ x
    dbias = dz.sum(axis=0)
    dx += dz @ _f64(w_router)
    return dict(dx=dx, dw_router=dw_router, dbias=dbias, dw1=dw1, dw3=dw3, dw2=dw2,
                dlogits=dz, dgate=dgate)


def lb_loss_grad(z, k, routing, alpha, lb_stopgrad_u=False):
    """d L_LB / d logits for the Section 3.3 loss alone (scale 1)."""
    z = _f64(z)
    T, E = z.shape
    kk = E if routing == ROUTE_SOFT else k
    idx = top_k_select(z, kk)
    g = gate_values(z, idx, routing)
    p_tok = full_softmax(z)
    _, u, p = lb_loss(dense_gates(idx, g, E), p_tok, alpha)
    dgate = np.zeros((T, kk), dtype=_F64)
    if not lb_stopgrad_u:
        dgate += alpha * E / T * p[idx.astype(np.int64)]
    return router_backward_dz(idx, g, p_tok, dgate, u, alpha, 1.0, routing)


# --------------------------------------------------------------------------------------
# Slice modes: the same definitions restricted to part of the output, so that full-size
# results can be checked in seconds.
# --------------------------------------------------------------------------------------

def moe_backward_token_slice(x, w_router, w1, w3, w2, dy, idx, gates, probs, u, p, tokens,
                             routing=ROUTE_TOPK, alpha=0.01, lb_grad_scale=1.0,
                             lb_stopgrad_u=False, keep=None):
    """dx, dlogits and dgate for the listed tokens only, given the routing of the whole batch
    (`keep`: the whole batch's capacity decisions, all kept when None)."""
    x = _f64(x)
    dy = _f64(dy)
    tok = np.asarray(tokens, dtype=np.int64)
    T = x.shape[0]
    E = np.asarray(w1).shape[0]
    idx = np.asarray(idx)
    g = _f64(gates)
    kk = idx.shape[1]
    keep = np.ones(idx.shape, dtype=bool) if keep is None else np.asarray(keep, dtype=bool)
    dx = np.zeros((len(tok), x.shape[1]), dtype=_F64)
    dgate = np.zeros((len(tok), kk), dtype=_F64)
    for slot in range(kk):
        for e in range(E):
            m = (idx[tok, slot] == e) & keep[tok, slot]
            if not np.any(m):
                continue
            xe = x[tok[m]]
            w1e, w3e, w2e = _f64(w1[e]), _f64(w3[e]), _f64(w2[e])
            y_e, h1, h3, a = swiglu_ffn(xe, w1e, w3e, w2e, return_hidden=True)
            dye = dy[tok[m]]
            dgate[m, slot] = np.sum(dye * y_e, axis=1)
            da = (g[tok[m], slot][:, None] * dye) @ w2e
            s = sigmoid(h1)
            dx[m] += (da * h3 * s * (1.0 + h1 * (1.0 - s))) @ w1e + (da * h1 * s) @ w3e
    if not lb_stopgrad_u:
        dgate += lb_grad_scale * alpha * E / T * _f64(p)[idx[tok].astype(np.int64)]
    dz = router_backward_dz(idx[tok], g[tok], _f64(probs)[tok], dgate, u, alpha, lb_grad_scale,
                            routing, batch_size=T)
    dx += dz @ _f64(w_router)
    return dict(dx=dx, dlogits=dz, dgate=dgate)


def router_wgrad_from_dz(x, dz):
    """dW_l = sum_t dz_t (outer) x_t  and  dbias = sum_t dz_t  over all tokens, from a supplied
    d(loss)/d(logits) array dz[T, E]: the last step of the router backward on its own, so that a
    full-size router gradient can be checked against the dz another implementation produced."""
    x = _f64(x)
    dz = _f64(dz)
    if dz.shape[0] != x.shape[0]:
        raise ValueError("dz and x must have one row per token")
    return dz.T @ x, dz.sum(axis=0)


def expert_wgrad_hidden_slice(x, w1, w3, w2, dy, idx, gates, e, hidden, keep=None):
    """dW1[e, J, :], dW3[e, J, :], dW2[e, :, J] for hidden units J, over all (kept) tokens of expert e.

    Uses da[t, J] = g_t * sum_c dY[t, c] W2[c, J], so the cost grows with |J| only.
    """
    x = _f64(x)
    dy = _f64(dy)
    J = np.asarray(hidden, dtype=np.int64)
    idx = np.asarray(idx)
    g = _f64(gates)
    d = x.shape[1]
    dw1 = np.zeros((len(J), d), dtype=_F64)
    dw3 = np.zeros((len(J), d), dtype=_F64)
    dw2 = np.zeros((d, len(J)), dtype=_F64)
    w1J, w3J, w2J = _f64(w1[e][J]), _f64(w3[e][J]), _f64(w2[e][:, J])
    keep = np.ones(idx.shape, dtype=bool) if keep is None else np.asarray(keep, dtype=bool)
    for slot in range(idx.shape[1]):
        m = (idx[:, slot] == e) & keep[:, slot]
        if not np.any(m):
            continue
        xe = x[m]
        h1 = xe @ w1J.T
        h3 = xe @ w3J.T
        s = sigmoid(h1)
        a = h1 * s * h3
        dout = g[m, slot][:, None] * dy[m]
        da = dout @ w2J
        dw2 += dout.T @ a
        dw1 += (da * h3 * s * (1.0 + h1 * (1.0 - s))).T @ xe
        dw3 += (da * h1 * s).T @ xe
    return dw1, dw3, dw2


# --------------------------------------------------------------------------------------
# Merge (Section 3.2: FFNs become the experts; every other parameter is averaged)
# --------------------------------------------------------------------------------------

def round_to_bf16(v):
    """Round float64 values to the nearest bfloat16 (ties to even), returned as float64."""
    v = _f64(v)
    out = np.zeros_like(v)
    nz = (v != 0) & np.isfinite(v)
    _, e = np.frexp(v[nz])                         # |v| = m * 2**e with 0.5 <= m < 1
    q_exp = np.maximum(e - 8, -133)                # bf16: 8 significant bits; subnormal quantum 2**-133
    out[nz] = np.ldexp(np.rint(np.ldexp(v[nz], -q_exp)), q_exp)
    out[~np.isfinite(v)] = v[~np.isfinite(v)]
    return out


def round_to_storage(v, dtype):
    if dtype == "bf16":
        return round_to_bf16(v)
    if dtype == "f32":
        return _f64(v).astype(np.float32).astype(_F64)
    raise ValueError(dtype)


def merge_mean(sources):
    """Uniform mean over the N models in float64, unrounded."""
    acc = np.zeros_like(_f64(sources[0]))
    for s in sources:
        acc = acc + _f64(s)
    return acc / len(sources)


def merge_average(sources, dtype):
    """Uniform mean over the N models in float64, rounded once to the storage type."""
    return round_to_storage(merge_mean(sources), dtype)


def merge_stack(sources):
    """Expert i of the MoE layer is model i's feed-forward tensor, unchanged."""
    return np.stack([np.asarray(s) for s in sources], axis=0)


FFN_STACK, FFN_SPLIT, FFN_BLEND = 0, 1, 2


def merge_ffn_layout(w1s, w3s, w2s, layout, chunks=1):
    """Expert tensors of one MoE layer from the N models' feed-forward matrices (lists of [F,d], [F,d],
    [d,F] arrays).  STACK: expert i = model i.  SPLIT (Section 3.3, "Splitting Experts"): every FF is cut
    into `chunks` pieces of d_ff/chunks hidden units, giving N*chunks experts.  BLEND ("Blending
    Experts"): every FF is cut into N pieces and expert n collects the n-th piece of every model."""
    N = len(w1s)
    F, d = np.asarray(w1s[0]).shape
    if layout == FFN_STACK:
        return merge_stack(w1s), merge_stack(w3s), merge_stack(w2s)
    C = chunks if layout == FFN_SPLIT else N
    if F % C:
        raise ValueError("d_ff must be divisible by the number of chunks")
    Fc = F // C
    piece = lambda i, c: (np.asarray(w1s[i])[c * Fc:(c + 1) * Fc], np.asarray(w3s[i])[c * Fc:(c + 1) * Fc],
                          np.asarray(w2s[i])[:, c * Fc:(c + 1) * Fc])
    o1, o3, o2 = [], [], []
    if layout == FFN_SPLIT:
        for i in range(N):
            for c in range(C):
                a, b, w = piece(i, c)
                o1.append(a); o3.append(b); o2.append(w)
    else:
        for n in range(N):
            parts = [piece(i, n) for i in range(N)]
            o1.append(np.concatenate([q[0] for q in parts], axis=0))
            o3.append(np.concatenate([q[1] for q in parts], axis=0))
            o2.append(np.concatenate([q[2] for q in parts], axis=1))
    return np.stack(o1), np.stack(o3), np.stack(o2)


def merge_models(models, dtype):
    """models: list of N dicts name -> array (same names/shapes).  Names containing '.ffn.'
    are stacked along a new leading expert axis; all others are averaged."""
    out = {}
    for name in models[0]:
        srcs = [m[name] for m in models]
        if ".ffn." in name:
            out[name] = merge_stack(srcs)
        else:
            out[name] = merge_average(srcs, dtype)
    return out


# --------------------------------------------------------------------------------------
# Parameter bookkeeping for a Llama-2-7B-shaped model (used to build the merge workload)
# --------------------------------------------------------------------------------------

def llama_like_param_shapes(n_layers, d_model, d_ff, vocab):
    """(name, shape) list: embeddings, per layer 4 attention matrices, 2 norms and the
    3 FFN matrices, final norm and output head."""
    shapes = [("tok_embeddings", (vocab, d_model))]
    for l in range(n_layers):
        for nm in ("wq", "wk", "wv", "wo"):
            shapes.append((f"layers.{l}.attn.{nm}", (d_model, d_model)))
        shapes.append((f"layers.{l}.attn_norm", (d_model,)))
        shapes.append((f"layers.{l}.ffn_norm", (d_model,)))
        shapes.append((f"layers.{l}.ffn.w1", (d_ff, d_model)))
        shapes.append((f"layers.{l}.ffn.w3", (d_ff, d_model)))
        shapes.append((f"layers.{l}.ffn.w2", (d_model, d_ff)))
    shapes.append(("norm", (d_model,)))
    shapes.append(("output", (vocab, d_model)))
    return shapes


def active_parameters(n_layers, d_model, d_ff, vocab, n_experts, k):
    """Parameters touched per token by the merged MoE model: all non-FFN parameters, the
    routers, and k of the n_experts feed-forward blocks in each layer."""
    ffn = 0
    other = 0
    for name, shp in llama_like_param_shapes(n_layers, d_model, d_ff, vocab):
        n = int(np.prod(shp))
        if ".ffn." in name:
            ffn += n
        else:
            other += n
    router = n_layers * n_experts * d_model
    return other + router + k * ffn
