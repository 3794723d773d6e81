"""Seeded synthetic inputs: model shapes, random-init weights, prompts, skip sets.

This module is the only code shared by the CPU oracle's tests and the CUDA
library's tests and benchmark.  It holds none of the method's arithmetic: it
draws numbers, scales the tensors the recipe says to scale, rounds to the
storage type and returns plain torch tensors.

Recipe (stand-in for trained LLaMA-2 weights and for dataset prompts, which
are not available offline):
  * every matrix ~ N(0, 0.02^2), one generator stream per tensor derived from
    a master seed; norm gains are 1;
  * the o_proj and down_proj of the layers the draft skips are multiplied by
    0.05 so that skipping them perturbs the residual stream only slightly;
  * for bf16 shapes the fp32 draw is rounded to bf16 (round-to-nearest-even);
    those bf16 values are the model;
  * prompts are uniform-random token ids in [0, vocab).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Sequence

import numpy as np
import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    dtype: str = "f32"  # "f32" or "bf16": storage type of weights and KV cache

    def params_per_layer(self) -> int:
        d, f = self.d_model, self.d_ffn
        return 4 * d * d + 3 * d * f

    def n_params(self) -> int:
        return self.n_layers * self.params_per_layer() + 2 * self.vocab * self.d_model


TINY = ModelShape("tiny-f32", 4, 256, 4, 64, 688, 2048, dtype="f32")
TINY_V64 = replace(TINY, name="tiny-f32-v64", vocab=64)
TINY_BF16 = replace(TINY, name="tiny-bf16", dtype="bf16")
LLAMA7B = ModelShape("llama2-7b-shape-bf16", 32, 4096, 32, 128, 11008, 32000, dtype="bf16")
LLAMA13B = ModelShape("llama2-13b-shape-bf16", 40, 5120, 40, 128, 13824, 32000, dtype="bf16")
# One 7B-shaped layer stack cut down to a few layers: same per-kernel shapes as
# LLAMA7B, small enough for the CPU oracle to finish in seconds.
LLAMA7B_4L = replace(LLAMA7B, name="llama2-7b-shape-4layers-bf16", n_layers=4)

# The 13B shape cut to two layers: d = 5120 (40 heads), FFN 13824, for shape coverage of the kernels.
LLAMA13B_2L = replace(LLAMA13B, name="llama2-13b-shape-2layers-bf16", n_layers=2)

MASTER_SEED = 20260205
PROMPT_SEED = 1234


def choose_skip_layers(n_layers: int, n_skip: int, how: str = "late", seed: int = MASTER_SEED) -> List[int]:
    """The layers whose output projections are down-scaled and which the draft skips.

    "late":   the n_skip layers just before the last one, L-1-n_skip .. L-2.  In a
              random-init stack the residual stream grows with depth, so late layers
              change it least; measured with the CPU oracle on the 7B shape (k=4) this
              set is accepted about 80% of the time against about 55% for "seeded".
    "seeded": the first n_skip entries of a seeded permutation of layers 1..L-2, sorted.
    The first and the last layer are never skipped.
    """
    if n_skip == 0:
        return []
    if n_skip > n_layers - 2:
        raise ValueError("cannot skip that many layers")
    if how == "late":
        return list(range(n_layers - 1 - n_skip, n_layers - 1))
    inner = np.arange(1, n_layers - 1)
    rng = np.random.RandomState(seed % (2**31))
    return sorted(int(x) for x in rng.permutation(inner)[:n_skip])


def keep_mask(n_layers: int, skip: Sequence[int]) -> np.ndarray:
    m = np.ones(n_layers, dtype=np.uint8)
    for l in skip:
        m[l] = 0
    return m


_TENSORS_PER_LAYER = ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down")


def _normal(shape, seed: int, device: str) -> torch.Tensor:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32) * 0.02


def _gain(d: int, seed: int, device: str, random_gains: bool) -> torch.Tensor:
    """RMSNorm gain: ones (the recipe), or uniform in [0.5, 1.5) for tests of the gain path."""
    if not random_gains:
        return torch.ones(d, device=device, dtype=torch.float32)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return torch.rand(d, generator=g, device=device, dtype=torch.float32) + 0.5


def make_weights(shape: ModelShape, skip: Sequence[int], seed: int = MASTER_SEED,
                 down_scale: float = 0.05, device: str = "cpu", random_gains: bool = False,
                 skip_ffn: Sequence[int] = None) -> Dict:
    """Random-init weights as a dict of torch tensors on `device`.

    Matrices are [out_features, in_features] row-major.  The draw happens on
    `device` (a CUDA generator and a CPU generator give different numbers for
    the same seed, so a test that needs the same model on both sides draws once
    and copies).  Storage dtype follows shape.dtype.  random_gains=True replaces the
    unit RMSNorm gains by seeded draws from [0.5, 1.5) (rounded to the storage type), so
    that a test can see whether every gain reaches the right column.  With skip_ffn given,
    the pruned blocks are chosen per sub-layer: o_proj is scaled in the layers of `skip`
    (attention blocks the draft drops), down_proj in the layers of `skip_ffn`.
    """
    st = torch.float32 if shape.dtype == "f32" else torch.bfloat16
    d, f, v = shape.d_model, shape.d_ffn, shape.vocab
    skip = set(int(s) for s in skip)
    skip_ffn = skip if skip_ffn is None else set(int(s) for s in skip_ffn)
    w: Dict = {"layers": []}
    w["tok_embed"] = _normal((v, d), seed * 1000 + 1, device).to(st)
    w["lm_head"] = _normal((v, d), seed * 1000 + 2, device).to(st)
    w["final_norm"] = _gain(d, seed * 1000 + 3, device, random_gains).to(st)
    dims = {"wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
            "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f)}
    for l in range(shape.n_layers):
        lw = {}
        for ti, name in enumerate(_TENSORS_PER_LAYER):
            t = _normal(dims[name], seed * 1000 + 10 + l * 16 + ti, device)
            if (l in skip and name == "wo") or (l in skip_ffn and name == "w_down"):
                t = t * down_scale
            lw[name] = t.to(st)
        lw["attn_norm"] = _gain(d, seed * 1000 + 10 + l * 16 + 8, device, random_gains).to(st)
        lw["ffn_norm"] = _gain(d, seed * 1000 + 10 + l * 16 + 9, device, random_gains).to(st)
        w["layers"].append(lw)
    return w


def weights_to(w: Dict, device: str) -> Dict:
    """Copy of a weight dict on another device (same values, same dtype)."""
    out = {"layers": []}
    for k, t in w.items():
        if k != "layers":
            out[k] = t.to(device)
    for lw in w["layers"]:
        out["layers"].append({k: t.to(device) for k, t in lw.items()})
    return out


def make_prompts(vocab: int, batch: int, prompt_len: int, seed: int = PROMPT_SEED) -> np.ndarray:
    """Uniform-random token ids, int32 [batch, prompt_len]; row b uses seed+b."""
    out = np.empty((batch, prompt_len), dtype=np.int32)
    for b in range(batch):
        rng = np.random.RandomState((seed + b) % (2**31))
        out[b] = rng.randint(0, vocab, size=prompt_len)
    return out
