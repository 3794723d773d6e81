"""GPU sampled decoding against the oracle: same Philox streams give the same tokens, and
the sampled distribution matches the target's exact softmax (vocabulary 64)."""
import numpy as np
import pytest
from scipy import stats

import synth_inputs as si
from oracle import sdfp_oracle as orc

from gpu_common import make_pair

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiny64():
    eng, m, _ = make_pair(si.TINY_V64, (1, 2), max_batch=8, k_max=6)
    yield eng, m
    eng.close()


def test_sampled_tokens_match_oracle(tiny64):
    """Same seed, same counters: the GPU draws what the oracle draws.  Both sides compute the
    probabilities in different precision, so a draw that lands within rounding of a CDF step may
    differ; such cases must be rare."""
    eng, m = tiny64
    prompt = si.make_prompts(64, 1, 16)
    T = 1.0 / 8.0
    same = total = 0
    for seed in range(40):
        out = eng.sdfp_generate(prompt, 4, 24, temperature=T, seed=seed)
        ref = orc.spec_generate(orc.CachedLM(m, max_seq=64), orc.CachedLM(m, [0, 3], max_seq=64),
                                prompt[0].tolist(), 4, 24, temperature=T, seed=seed)
        total += 1
        if out.tokens[0] == ref.tokens:
            same += 1
            assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]
        ar = eng.sdfp_generate(prompt, 0, 24, temperature=T, seed=seed)
        ar_ref = orc.ar_generate(orc.CachedLM(m, max_seq=64), prompt[0].tolist(), 24, temperature=T, seed=seed)
        total += 1
        same += (ar.tokens[0] == ar_ref.tokens)
    assert same >= total - 2


def _merge_small(obs, exp, floor=5.0):
    big = exp >= floor
    o_, e_ = list(obs[big]), list(exp[big])
    if (~big).any():
        o_.append(obs[~big].sum())
        e_.append(exp[~big].sum())
    return np.array(o_), np.array(e_)


def test_chi_square_on_gpu(tiny64):
    """1e5 sampled speculative generations of two tokens (8 sequences per call share the
    prompt; the Philox counter carries the sequence index): y1 and (y1, y2) against the
    target's exact distribution from the oracle."""
    eng, m = tiny64
    prompt = si.make_prompts(64, 1, 16)[0]
    T = 1.0 / 8.0
    prompts = np.tile(prompt, (8, 1))
    n_calls = 12500
    c1 = np.zeros(64)
    c2 = np.zeros((64, 64))
    n_rej = 0
    for seed in range(n_calls):
        out = eng.sdfp_generate(prompts, 2, 2, temperature=T, seed=seed)
        for b in range(8):
            c1[out.tokens[b][0]] += 1
            c2[out.tokens[b][0], out.tokens[b][1]] += 1
        n_rej += int((out.stats[0, :, 1] < 2).sum())
    n = n_calls * 8
    pl = prompt.tolist()
    p1 = orc.softmax_T(orc.forward_nocache(m, pl)[-1], T).numpy()
    p2 = np.stack([orc.softmax_T(orc.forward_nocache(m, pl + [a])[-1], T).numpy() for a in range(64)])
    assert n_rej > 0.05 * n
    ob, ex = _merge_small(c1, p1 * n)
    assert stats.chisquare(ob, ex).pvalue > 1e-3
    ob, ex = _merge_small(c2.ravel(), (p1[:, None] * p2).ravel() * n)
    assert stats.chisquare(ob, ex).pvalue > 1e-3


def test_sampling_draft_equal_target_accepts_all(tiny64):
    eng, m = tiny64
    eng.sdfp_set_draft_layers([1, 1, 1, 1])
    try:
        out = eng.sdfp_generate(si.make_prompts(64, 1, 16), 4, 20, temperature=1.0, seed=11)
    finally:
        eng.sdfp_set_draft_layers(si.keep_mask(4, (1, 2)))
    assert (out.stats[:, 0, 1] == 4).all()


# ---- vocabularies where a thread of the draw owns several elements ---------------------------------

def test_sampled_tokens_match_oracle_vocab_2048():
    """Vocabulary 2048 with 1024 threads: every thread sums a two-element segment, the scan runs
    over non-trivial totals and the owner walks its segment.  Same rule as at vocabulary 64."""
    eng, m, _ = make_pair(si.TINY, (1, 2), max_seq=64, k_max=6)
    try:
        prompt = si.make_prompts(m.vocab, 1, 16)
        T = 1.0 / 8.0
        same = total = 0
        for seed in range(40):
            out = eng.sdfp_generate(prompt, 4, 24, temperature=T, seed=seed)
            ref = orc.spec_generate(orc.CachedLM(m, max_seq=64), orc.CachedLM(m, [0, 3], max_seq=64),
                                    prompt[0].tolist(), 4, 24, temperature=T, seed=seed)
            total += 1
            if out.tokens[0] == ref.tokens:
                same += 1
                assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]
            ar = eng.sdfp_generate(prompt, 0, 24, temperature=T, seed=seed)
            ar_ref = orc.ar_generate(orc.CachedLM(m, max_seq=64), prompt[0].tolist(), 24, temperature=T, seed=seed)
            total += 1
            same += (ar.tokens[0] == ar_ref.tokens)
        assert same >= total - 2
    finally:
        eng.close()


def test_sampled_tokens_match_oracle_vocab_32000():
    """The sampled configuration's real vocabulary and draft length (V = 32000, k = 6, temperature
    1) on the 7B layer shapes: 32-element segments per thread.  Tokens and acceptance counts
    against the oracle's loop, seed by seed."""
    shape = si.LLAMA7B_4L
    eng, m, _ = make_pair(shape, (1, 2), max_seq=64, k_max=6, draw_device="cuda:0")
    try:
        prompt = si.make_prompts(shape.vocab, 1, 12, seed=31)
        same = total = 0
        accepted = drafted = 0
        for seed in range(6):
            out = eng.sdfp_generate(prompt, 6, 14, temperature=1.0, seed=seed)
            ref = orc.spec_generate(orc.CachedLM(m, max_seq=64), orc.CachedLM(m, [0, 3], max_seq=64),
                                    prompt[0].tolist(), 6, 14, temperature=1.0, seed=seed)
            total += 1
            accepted += int(out.stats[:, 0, 1].sum())
            drafted += int(out.stats[:, 0, 0].sum())
            if out.tokens[0] == ref.tokens:
                same += 1
                assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]
                assert out.stats[:, 0, 2].tolist() == [r.committed for r in ref.rounds]
        assert same >= total - 1
        assert 0 < accepted < drafted                  # both outcomes of the accept test occurred
    finally:
        eng.close()


def test_sampled_decoding_on_the_dense_path():
    """A bf16 context too wide for the whole-pass kernel (4 sequences x 5 rows) decodes on the tcgen05
    path: sampled speculative decoding of a batch against the oracle, sequence by sequence (the
    sequence index is part of the Philox counter), and the autoregressive sampler likewise."""
    # vocabulary 64: with bf16 logits (error ~1e-4, times 1/T) and thousands of CDF steps a draw would
    # land within rounding of a step in a fifth of the streams; with 64 steps it practically never does
    from dataclasses import replace
    shape = replace(si.TINY_V64, name="tiny-bf16-v64", dtype="bf16")
    eng, m, _ = make_pair(shape, (1, 2), max_seq=96, max_batch=4, k_max=4)
    try:
        prompts = si.make_prompts(m.vocab, 4, 20, seed=33)
        T = 1.0 / 8.0
        same = total = 0
        for seed in range(6):
            out = eng.sdfp_generate(prompts, 4, 16, temperature=T, seed=seed)
            ar = eng.sdfp_generate(prompts, 0, 16, temperature=T, seed=seed)
            for b in range(4):
                ref = orc.spec_generate(orc.CachedLM(m, max_seq=96), orc.CachedLM(m, [0, 3], max_seq=96),
                                        prompts[b].tolist(), 4, 16, temperature=T, seed=seed, seq=b)
                ar_ref = orc.ar_generate(orc.CachedLM(m, max_seq=96), prompts[b].tolist(), 16, temperature=T, seed=seed, seq=b)
                total += 2
                same += (out.tokens[b] == ref.tokens) + (ar.tokens[b] == ar_ref.tokens)
                if out.tokens[b] == ref.tokens:
                    acc_b = [int(a) for a, d in zip(out.stats[:, b, 1], out.stats[:, b, 0]) if d > 0]
                    assert acc_b == [r.accepted for r in ref.rounds]
        assert same >= total - 3
    finally:
        eng.close()
