"""FIT layer scores of Algorithm 1, Stage A, on the CPU.  TEST INFRASTRUCTURE.

T_l = (1/N) Σ_i ‖∇_{θ_l} f(z_i, θ)‖²  (the empirical-Fisher trace of layer l, the
paper's per-layer score), and the FIT form Ω_l = Tr(I(θ_l)) · E[δθ_l²] (the
layer-wise FIT equation) with the perturbation of *removing* the layer read
as δθ = −θ, i.e. E[δθ_t²] = mean(θ_t²) per tensor t of the layer:

    FIT_l = Σ_{t ∈ layer l} T_t · mean(θ_t²).

The paper then assumes the perturbation variance to be the same for every
layer and ranks by T_l alone; both numbers are returned.  Gradients come from
reverse-mode differentiation (torch autograd) of the no-cache forward; the
tests check them against central finite differences.

f(z_i, θ) is the mean next-token cross-entropy over one calibration sequence
(one sequence = one sample = one minibatch, so the per-sample form of the
score and the minibatch loop of Algorithm 1 coincide).
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple

import torch

from .sdfp_oracle import Model, forward_nocache

LAYER_TENSORS = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "ffn_norm")


def sequence_loss(m: Model, tokens: Sequence[int]) -> torch.Tensor:
    """Mean cross-entropy of token t+1 under the logits at position t."""
    logits = forward_nocache(m, tokens[:-1])
    tgt = torch.tensor(list(tokens[1:]), dtype=torch.long)
    logp = torch.log_softmax(logits, dim=-1)
    return -logp[torch.arange(len(tgt)), tgt].mean()


def grad_model(m: Model, dtype=torch.float64) -> Model:
    """A copy of the model whose tensors are leaves that require gradients."""
    w = {"layers": []}
    for k, t in m.w.items():
        if k != "layers":
            w[k] = t.detach().to(dtype).clone().requires_grad_(True)
    for lw in m.w["layers"]:
        w["layers"].append({k: t.detach().to(dtype).clone().requires_grad_(True) for k, t in lw.items()})
    return Model(w, m.n_layers, m.d_model, m.n_heads, m.head_dim, m.d_ffn, m.vocab,
                 m.rms_eps, m.rope_theta, kv_bf16=False, dtype=dtype)


def fit_scores(m: Model, calib: Sequence[Sequence[int]], dtype=torch.float64) -> Tuple[List[float], List[float]]:
    """Returns (T_l, FIT_l) for l = 0..L−1 over the calibration sequences."""
    gm = grad_model(m, dtype)
    L = gm.n_layers
    sq = [{t: 0.0 for t in LAYER_TENSORS} for _ in range(L)]
    for seq in calib:
        for lw in gm.w["layers"]:
            for t in lw.values():
                t.grad = None
        loss = sequence_loss(gm, seq)
        loss.backward()
        for l in range(L):
            for t in LAYER_TENSORS:
                g = gm.w["layers"][l][t].grad
                sq[l][t] += float((g * g).sum())
    N = len(calib)
    T = [sum(sq[l].values()) / N for l in range(L)]
    FIT = []
    for l in range(L):
        s = 0.0
        for t in LAYER_TENSORS:
            theta = gm.w["layers"][l][t].detach()
            s += (sq[l][t] / N) * float((theta * theta).mean())
        FIT.append(s)
    return T, FIT


def prune_set(scores: Sequence[float], ratio: float) -> List[int]:
    """Algorithm 1: sort ascending, take the ⌊r·L⌋ lowest."""
    L = len(scores)
    order = sorted(range(L), key=lambda l: (scores[l], l))
    return sorted(order[: int(ratio * L)])
