"""Pins of the FIT oracle (Algorithm 1, Stage A): gradients against central finite
differences, order invariance, and the ranking the synthetic recipe must produce."""
import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import fit
from oracle import sdfp_oracle as o


def test_gradients_match_finite_differences():
    shape = si.ModelShape("fd", 2, 32, 2, 16, 40, 50)
    w = si.make_weights(shape, [])
    # larger weights than the recipe's so that every gradient is well above rounding
    for lw in w["layers"]:
        for k in lw:
            if k.startswith("w"):
                lw[k] *= 10.0
    gm = fit.grad_model(o.Model.from_shape(shape, w), torch.float64)
    seq = si.make_prompts(shape.vocab, 1, 12, seed=7)[0].tolist()
    fit.sequence_loss(gm, seq).backward()
    rng = np.random.RandomState(0)
    eps = 1e-5
    for l in range(2):
        for name in fit.LAYER_TENSORS:
            t = gm.w["layers"][l][name]
            flat = t.detach().view(-1)
            for idx in rng.choice(flat.numel(), size=20, replace=False):
                old = float(flat[idx])
                with torch.no_grad():
                    flat[idx] = old + eps
                    fp = float(fit.sequence_loss(gm, seq))
                    flat[idx] = old - eps
                    fm = float(fit.sequence_loss(gm, seq))
                    flat[idx] = old
                fd = (fp - fm) / (2 * eps)
                an = float(t.grad.view(-1)[idx])
                assert an == pytest.approx(fd, rel=1e-3, abs=1e-9), (l, name, idx)


def test_loss_of_uniform_model_is_log_vocab():
    """With a zero lm-head every token is equally likely: f = log V exactly."""
    shape = si.ModelShape("u", 1, 16, 1, 16, 24, 37)
    w = si.make_weights(shape, [])
    w["lm_head"].zero_()
    m = o.Model.from_shape(shape, w, dtype=torch.float64)
    assert float(fit.sequence_loss(m, [1, 2, 3, 4, 5])) == pytest.approx(np.log(37), rel=1e-12)


def test_c1_downscaled_layers_rank_least_sensitive():
    """Layers {1,2} of the tiny config have o_proj/down_proj scaled by 0.05: FIT must
    rank them lowest, so Algorithm 1 with r = 0.5 selects exactly them."""
    w = si.make_weights(si.TINY, (1, 2))
    m = o.Model.from_shape(si.TINY, w)
    calib = [row.tolist() for row in si.make_prompts(si.TINY.vocab, 8, 32, seed=99)]
    T, FIT = fit.fit_scores(m, calib)
    assert fit.prune_set(FIT, 0.5) == [1, 2]
    assert max(FIT[1], FIT[2]) < 0.2 * min(FIT[0], FIT[3])
    # order of the calibration samples does not matter
    T2, FIT2 = fit.fit_scores(m, calib[::-1])
    assert T2 == pytest.approx(T, rel=1e-10) and FIT2 == pytest.approx(FIT, rel=1e-10)
    # ⌊rL⌋ with r = 0.3, L = 4 -> one layer
    assert len(fit.prune_set(FIT, 0.3)) == 1


def test_prune_set_floor_and_ascending():
    assert fit.prune_set([5.0, 1.0, 3.0, 0.5, 9.0], 0.4) == [1, 3]
    assert fit.prune_set([5.0, 1.0, 3.0, 0.5, 9.0], 0.39) == [3]
    assert fit.prune_set([1.0, 1.0, 1.0], 0.34) == [0]
