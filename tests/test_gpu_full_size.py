"""Parity at the full size of the benchmark workload (7B shape, 32 layers, 12 skipped, bf16), in the
launch configurations the benchmark times: one cooperative launch of the whole-pass kernel per pass
on every SM (batch 1), and the dense path's launches per layer (batch 8).  The oracle cannot decode hundreds of tokens at this size, so it checks sampled
outputs: the logits of a short prompt through all 32 layers and through the draft's 20 layers, and
every one of the first tokens the library generates after the benchmark's 512-token prompt
(teacher-forced, near-ties reported).  What holds at any length is checked on the whole run:
speculative greedy output equals autoregressive output, acceptance counts are consistent."""
import numpy as np
import pytest

import synth_inputs as si
from oracle import sdfp_oracle as orc

from gpu_common import check_stream_against_oracle, make_pair, rel_l2

pytestmark = pytest.mark.gpu

N_SKIP, K, PROMPT_LEN, N_NEW = 12, 4, 512, 24


@pytest.fixture(scope="module")
def c2():
    shape = si.LLAMA7B
    skip = si.choose_skip_layers(shape.n_layers, N_SKIP)
    eng, m, _ = make_pair(shape, skip, max_seq=PROMPT_LEN + 256 + 16, k_max=8, draw_device="cuda:0")
    yield eng, m, skip
    eng.close()


@pytest.fixture(scope="module")
def c5(c2):
    """The same weights (same seeds) in a context of 8 sequence slots, k up to 8: 72-row verify
    passes, every pass on the dense path (the batch-8 configuration of the benchmark's sweep)."""
    import paper_2602_05499_b200 as pkg
    _, m, skip = c2
    shape = si.LLAMA7B
    w = si.make_weights(shape, skip, device="cuda:0")
    eng = pkg.Sdfp(shape, w, max_seq=PROMPT_LEN + 64 + 16, max_batch=8, k_max=8)
    eng.sdfp_set_draft_layers(si.keep_mask(shape.n_layers, skip))
    del w
    yield eng, m, skip
    eng.close()


def test_full_size_logits(c2):
    """Rows 0..19 of a prompt: a 16-row pass (two column groups) and a 4-row pass, target and draft."""
    eng, m, skip = c2
    toks = si.make_prompts(m.vocab, 1, 20, seed=77)[0].tolist()
    got = eng.sdfp_forward_logits(toks, 0)
    ref = orc.forward_nocache(m, toks).detach().numpy()
    assert rel_l2(got, ref) < 1e-2
    assert max(rel_l2(got[r], ref[r]) for r in range(len(toks))) < 1e-2
    kept = orc.keep_layers(m.n_layers, skip)
    got_d = eng.sdfp_forward_logits(toks, 0, draft=True)
    ref_d = orc.forward_nocache(m, toks, kept).detach().numpy()
    assert rel_l2(got_d, ref_d) < 1e-2
    # a single-row pass (one column group, the configuration of a decode step) gives the same bits
    one = eng.sdfp_forward_logits(toks[:1], 0)
    assert np.array_equal(one.view(np.uint32), got[:1].view(np.uint32))


def test_full_size_greedy_stream(c2):
    """The benchmark's prompt length; the first tokens are checked one by one against the oracle."""
    eng, m, skip = c2
    prompts = si.make_prompts(m.vocab, 1, PROMPT_LEN, seed=si.PROMPT_SEED)
    out = eng.sdfp_generate(prompts, K, 256)
    ar = eng.sdfp_generate(prompts, 0, 256)
    assert out.tokens == ar.tokens                      # lossless, bit for bit, over the whole run
    st = out.stats[:out.n_rounds, 0]
    assert (st[:, 1] <= st[:, 0]).all() and (st[:, 0] <= K).all()
    assert int(st[:, 2].sum()) == 256                   # committed tokens add up to what was asked
    assert ((st[:, 2] == st[:, 1] + 1) | (np.arange(out.n_rounds) == out.n_rounds - 1)).all()
    reported = check_stream_against_oracle(m, prompts[0].tolist(), out.tokens[0][:N_NEW])
    assert len(reported) <= 2, reported


def test_full_size_batch8_dense_path(c2, c5):
    """Batch 8 at full size: the dense path's logits against the oracle (target and draft), and
    against the whole-pass kernel's on the same weights; speculative == autoregressive for all eight
    sequences over the whole run, one sequence equals its solo run, and the first tokens of one
    sequence are checked one by one against the oracle."""
    eng1, m, skip = c2
    eng, _, _ = c5
    toks = si.make_prompts(m.vocab, 1, 20, seed=77)[0].tolist()
    got = eng.sdfp_forward_logits(toks, 0)
    ref = orc.forward_nocache(m, toks).detach().numpy()
    assert max(rel_l2(got[r], ref[r]) for r in range(len(toks))) < 1e-2
    got_d = eng.sdfp_forward_logits(toks, 0, draft=True)
    ref_d = orc.forward_nocache(m, toks, orc.keep_layers(m.n_layers, skip)).detach().numpy()
    assert max(rel_l2(got_d[r], ref_d[r]) for r in range(len(toks))) < 1e-2
    # the two arithmetic paths against each other: different summation orders and K/V rounded from values
    # that differ in their last bits, over 32 layers (each is within 1e-2 of the oracle)
    assert rel_l2(got, eng1.sdfp_forward_logits(toks, 0)) < 5e-3
    prompts = si.make_prompts(m.vocab, 8, PROMPT_LEN, seed=si.PROMPT_SEED + 1)
    for k in (4, 8):
        out = eng.sdfp_generate(prompts, k, 48)
        ar = eng.sdfp_generate(prompts, 0, 48)
        assert out.tokens == ar.tokens
        st = out.stats[:out.n_rounds]
        assert (st[:, :, 1] <= st[:, :, 0]).all() and (st[:, :, 0] <= k).all()
        assert (st[:, :, 2].sum(axis=0) == 48).all()
    assert eng.sdfp_generate(prompts[5:6], 4, 48).tokens[0] == out.tokens[5]
    reported = check_stream_against_oracle(m, prompts[2].tolist(), out.tokens[2][:8])
    assert len(reported) <= 1, reported
