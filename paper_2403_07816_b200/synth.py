"""Seeded synthetic inputs shaped like the paper's Llama-2-7B MoE-finetuning workload.

This module only draws random tensors (and names parameter shapes).  It contains none of the
layer's arithmetic, so both the CUDA path and the CPU checker can be fed from it.

Value distributions: token activations x ~ N(0, 1); router, W1, W3, W2 ~ N(0, 0.02^2);
upstream gradient dY ~ N(0, 1); all i.i.d.  A tensor is drawn in fp32 from a
`torch.Generator` seeded with (seed, tensor id) on the requested device and then rounded
to the storage dtype, so a run is reproducible on a given device type.
"""
from __future__ import annotations

import torch

WEIGHT_STD = 0.02

_TENSOR_IDS = {"x": 1, "w_router": 2, "w1": 3, "w3": 4, "w2": 5, "dy": 6}

# Router bias on expert 0 that makes it the first choice of about 70 % of tokens when the
# other logits are i.i.d. N(0, 0.02^2 * 4096) (d_model = 4096, x ~ N(0,1)).
SKEW_BIAS_EXPERT0 = 1.9


def _gen(seed: int, tensor_id: int, layer: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((int(seed) * 1000003 + int(layer)) * 101 + int(tensor_id))
    return g


def normal(shape, std, seed, tensor_id, dtype, device="cpu", layer=0):
    g = _gen(seed, tensor_id, layer, device)
    t = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
    if std != 1.0:
        t.mul_(std)
    return t.to(dtype).contiguous()


def moe_inputs(T, d_model, d_ff, E, seed, dtype=torch.float32, device="cpu", layer=0,
               with_dy=True):
    """Inputs of one MoE feed-forward layer: x[T,d], w_router[E,d], w1/w3[E,F,d], w2[E,d,F], dy[T,d]."""
    out = {
        "x": normal((T, d_model), 1.0, seed, _TENSOR_IDS["x"], dtype, device, layer),
        "w_router": normal((E, d_model), WEIGHT_STD, seed, _TENSOR_IDS["w_router"], dtype, device, layer),
        "w1": normal((E, d_ff, d_model), WEIGHT_STD, seed, _TENSOR_IDS["w1"], dtype, device, layer),
        "w3": normal((E, d_ff, d_model), WEIGHT_STD, seed, _TENSOR_IDS["w3"], dtype, device, layer),
        "w2": normal((E, d_model, d_ff), WEIGHT_STD, seed, _TENSOR_IDS["w2"], dtype, device, layer),
    }
    if with_dy:
        out["dy"] = normal((T, d_model), 1.0, seed, _TENSOR_IDS["dy"], dtype, device, layer)
    return out


def gumbel_noise(T, E, seed, device="cpu", layer=0):
    """Standard Gumbel noise G = -log(-log(U)), U ~ Uniform(0,1), fp32 [T, E]: the random numbers that
    Sample Top-1 routing draws; they are an input of the layer."""
    g = _gen(seed, 7, layer, device)
    u = torch.rand((T, E), generator=g, device=device, dtype=torch.float32).clamp_(1e-7, 1.0 - 1e-7)
    return (-torch.log(-torch.log(u))).contiguous()


def skew_bias(E, device="cpu"):
    b = torch.zeros(E, dtype=torch.float32, device=device)
    b[0] = SKEW_BIAS_EXPERT0
    return b


def llama_like_param_shapes(n_layers, d_model, d_ff, vocab):
    """(name, shape) of every parameter tensor; names containing '.ffn.' are feed-forward
    matrices (stacked by the merge), all others are averaged."""
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


def expert_models(n_models, n_layers, d_model, d_ff, vocab, seed, dtype=torch.float32,
                  device="cpu", names=None):
    """N parameter sets of the same architecture (the separately trained expert LLMs).
    `names` optionally restricts generation to some tensors (the big workload is sampled)."""
    shapes = llama_like_param_shapes(n_layers, d_model, d_ff, vocab)
    models = []
    for m in range(n_models):
        params = {}
        for tid, (name, shp) in enumerate(shapes):
            if names is not None and name not in names:
                continue
            params[name] = normal(shp, WEIGHT_STD, seed, 100 + tid, dtype, device, layer=m)
        models.append(params)
    return models


def to_f64_numpy(t: torch.Tensor):
    """Exact conversion of a stored tensor to float64 numpy (for the CPU checker)."""
    return t.detach().to("cpu").to(torch.float64).numpy()
