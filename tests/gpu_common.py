"""Helpers shared by the GPU parity tests: build a library context and an oracle on
the same seeded weights, and compare a GPU token stream with the oracle step by step."""
from __future__ import annotations

import numpy as np
import torch

import paper_2602_05499_b200 as pkg
import synth_inputs as si
from oracle import sdfp_oracle as orc


def make_pair(shape, skip, max_seq=160, max_batch=1, k_max=8, flags=0, eos_id=-1, draw_device="cpu",
              random_gains=False):
    """(library context, oracle Model, weights) on the same weights."""
    pkg.build_library()
    w = si.make_weights(shape, skip, device=draw_device, random_gains=random_gains)
    w_gpu = si.weights_to(w, "cuda:0")
    w_cpu = si.weights_to(w, "cpu")
    eng = pkg.Sdfp(shape, w_gpu, max_seq=max_seq, max_batch=max_batch, k_max=k_max, flags=flags, eos_id=eos_id)
    eng.sdfp_set_draft_layers(si.keep_mask(shape.n_layers, skip))
    del w_gpu
    return eng, orc.Model.from_shape(shape, w_cpu), w_cpu


def rel_l2(a, b) -> float:
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / np.linalg.norm(b))


def check_stream_against_oracle(m, prompt, gpu_tokens, gap_tol=1e-2, layers=None):
    """Teacher-force the oracle along the GPU's tokens: at every step the GPU's token must be
    the oracle's argmax, unless the oracle's logit of the GPU token is within gap_tol of its
    maximum (a near-tie, which is reported).  Returns the list of reported steps."""
    seq = list(prompt) + list(gpu_tokens)
    logits = orc.forward_nocache(m, seq[:-1], layers)
    P = len(prompt)
    reported = []
    for t, tok in enumerate(gpu_tokens):
        row = logits[P - 1 + t]
        best = orc.argmax_lowest(row)
        if tok != best:
            gap = float(row[best] - row[tok])
            assert gap < gap_tol, f"step {t}: GPU token {tok} vs oracle {best}, logit gap {gap:.4g}"
            reported.append((t, tok, best, gap))
    return reported
