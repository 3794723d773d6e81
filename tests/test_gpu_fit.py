"""Stage A of Algorithm 1 on the GPU (sdfp_fit_scores) against the CPU oracle's FIT scores, which
are themselves pinned by finite differences (tests/test_oracle_fit.py)."""
import numpy as np
import pytest
import torch

import paper_2602_05499_b200 as pkg
import synth_inputs as si
from oracle import fit
from oracle import sdfp_oracle as orc

pytestmark = pytest.mark.gpu


def _both(shape, w, calib):
    pkg.build_library()
    got_T, got_F = pkg.sdfp_fit_scores(shape, si.weights_to(w, "cuda:0"), calib)
    m = orc.Model.from_shape(shape, si.weights_to(w, "cpu"))
    ref_T, ref_F = fit.fit_scores(m, [list(map(int, r)) for r in calib])
    return got_T, got_F, ref_T, ref_F


def test_fit_scores_small_model_with_large_gradients():
    """The finite-difference test's model (weights x 10, so that every tensor's gradient is well
    above rounding), odd sizes: 2 layers, d 32, 2 heads x 16, FFN 40, vocabulary 50; sequences of
    12 tokens.  Every layer's trace and FIT value within 1e-3 of the fp64 oracle."""
    shape = si.ModelShape("fd", 2, 32, 2, 16, 40, 50)
    w = si.make_weights(shape, [], random_gains=True)
    for lw in w["layers"]:
        for k in lw:
            if k.startswith("w"):
                lw[k] *= 10.0
    calib = si.make_prompts(shape.vocab, 3, 12, seed=7)
    got_T, got_F, ref_T, ref_F = _both(shape, w, calib)
    assert got_T == pytest.approx(ref_T, rel=1e-3)
    assert got_F == pytest.approx(ref_F, rel=1e-3)


@pytest.mark.parametrize("shape", [si.TINY, si.TINY_BF16])
def test_fit_scores_tiny_config_and_ranking(shape):
    """The tiny configuration (fp32 and bf16 storage), 8 calibration sequences of 32 tokens: scores
    against the oracle, the two down-scaled layers rank lowest (Algorithm 1 with r = 0.5 selects
    exactly them), and the result does not depend on the order of the calibration set."""
    w = si.make_weights(shape, (1, 2))
    calib = si.make_prompts(shape.vocab, 8, 32, seed=99)
    got_T, got_F, ref_T, ref_F = _both(shape, w, calib)
    assert got_T == pytest.approx(ref_T, rel=2e-3)
    assert got_F == pytest.approx(ref_F, rel=2e-3)
    assert fit.prune_set(got_F, 0.5) == [1, 2]
    assert max(got_F[1], got_F[2]) < 0.2 * min(got_F[0], got_F[3])
    again_T, again_F = pkg.sdfp_fit_scores(shape, si.weights_to(w, "cuda:0"), calib[::-1].copy())
    assert again_T == pytest.approx(got_T, rel=1e-12) and again_F == pytest.approx(got_F, rel=1e-12)
    same_T, _ = pkg.sdfp_fit_scores(shape, si.weights_to(w, "cuda:0"), calib)
    assert same_T == got_T                                   # run to run: bit-identical


def test_fit_scores_drive_the_draft_mask():
    """Stage A feeding Stage B: the prune set chosen from the GPU scores is handed to
    sdfp_set_draft_layers and the speculative output stays the target's."""
    shape = si.TINY
    w = si.make_weights(shape, (1, 2))
    calib = si.make_prompts(shape.vocab, 8, 32, seed=99)
    _, F = pkg.sdfp_fit_scores(shape, si.weights_to(w, "cuda:0"), calib)
    skip = fit.prune_set(F, 0.5)
    assert skip == [1, 2]
    eng = pkg.Sdfp(shape, si.weights_to(w, "cuda:0"), max_seq=128, k_max=4)
    try:
        eng.sdfp_set_draft_layers(si.keep_mask(shape.n_layers, skip))
        prompt = si.make_prompts(shape.vocab, 1, 16)
        out = eng.sdfp_generate(prompt, 4, 32)
        assert out.tokens == eng.sdfp_generate(prompt, 0, 32).tokens
        assert out.acceptance_rate > 0.15
    finally:
        eng.close()


def test_fit_scores_rejects_bad_arguments():
    shape = si.TINY
    w = si.weights_to(si.make_weights(shape, (1, 2)), "cuda:0")
    with pytest.raises(pkg.SdfpError):
        pkg.sdfp_fit_scores(shape, w, np.full((2, 8), shape.vocab, dtype=np.int32))     # token out of range
    with pytest.raises(pkg.SdfpError):
        pkg.sdfp_fit_scores(shape, w, np.zeros((2, 1), dtype=np.int32))                 # nothing to predict
