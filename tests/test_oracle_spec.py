"""Pins of the oracle's decoding loops: scripted models whose answer is known by
construction, closed-form special cases, exact losslessness identities and a
chi-square test of the sampled distribution against exact enumeration."""
import math

import numpy as np
import pytest
import torch
from scipy import stats

import synth_inputs as si
from oracle import philox
from oracle import sdfp_oracle as o


# ---------------------------------------------------------------------------
# scripted language models: next-token logits are a table lookup on the last
# token, and the object checks the cache discipline of whoever drives it
# ---------------------------------------------------------------------------

class ScriptedLM:
    """next = table[last token]; logits one-hot-ish.  Records what sits at each cache
    position and insists that every feed extends a prefix that is really cached."""

    def __init__(self, table, vocab, truth=None):
        self.table, self.vocab = table, vocab
        self.cache = []           # token held at each position
        self.rows = 0
        self.calls = []

    def feed(self, tokens, start):
        assert start <= len(self.cache), "feed would leave a hole in the cache"
        self.cache = self.cache[:start] + [int(t) for t in tokens]
        self.rows += len(tokens)
        self.calls.append((start, len(tokens)))
        out = torch.full((len(tokens), self.vocab), -1.0)
        for r, t in enumerate(tokens):
            out[r, self.table[int(t)]] = 1.0
        return out


def _chain(vocab, wrong_at=()):
    """Target: next = (t+1) mod V.  A draft that errs on the listed tokens."""
    tgt = [(t + 1) % vocab for t in range(vocab)]
    drf = list(tgt)
    for t in wrong_at:
        drf[t] = (t + 2) % vocab
    return tgt, drf


def test_scripted_counts_and_cache_discipline():
    V, k = 50, 4
    tgt_t, drf_t = _chain(V, wrong_at=(7, 8, 20))
    target, draft = ScriptedLM(tgt_t, V), ScriptedLM(drf_t, V)
    prompt = [0, 1, 2, 3]
    res = o.spec_generate(target, draft, prompt, k, 30)
    assert res.tokens == [(4 + i) % V for i in range(30)]        # the target's chain, exactly
    # Worked by hand: the draft errs when its *input* token is 7, 8 or 20.
    # round 1: n=4, last=3, drafts 4,5,6,7 all right -> j=4, commit 4..8   (8 = bonus)
    # round 2: last=8, draft(8) wrong -> j=0, commit 9
    # round 3: last=9, drafts 10,11,12,13 -> j=4, commit 10..14
    # round 4: last=14, drafts 15..18 -> j=4, commit 15..19
    # round 5: last=19, drafts 20 ok, draft(20) wrong -> j=1, commit 20,21
    # round 6: last=21, 22..25 -> j=4, commit 22..26
    # round 7: last=26, 27..30 -> j=4, commit 27..31
    # round 8: last=31, 32..35 -> j=4, but only 2 tokens of room remain
    acc = [r.accepted for r in res.rounds]
    com = [r.committed for r in res.rounds]
    assert acc == [4, 0, 4, 4, 1, 4, 4, 4]
    assert com == [5, 1, 5, 5, 2, 5, 5, 2]
    assert all(r.drafted == k for r in res.rounds)
    assert res.acceptance_rate == pytest.approx(25 / 32)
    # the target is called once for the prompt and once per round with k+1 rows
    assert target.calls[0] == (0, 3)
    assert all(c[1] == k + 1 for c in target.calls[1:])
    # the draft's first call of a round feeds 2 rows exactly after a fully accepted round
    firsts = [c for c in draft.calls[1:] if c[1] != 1 or True]
    # positions fed to the draft are always backed by cached committed tokens (asserted inside feed)


def test_scripted_draft_two_rows_after_full_accept():
    V, k = 40, 3
    tgt_t, drf_t = _chain(V)
    target, draft = ScriptedLM(tgt_t, V), ScriptedLM(drf_t, V)
    res = o.spec_generate(target, draft, [5, 6], k, 12)
    assert res.tokens == [7 + i for i in range(12)]
    assert [r.accepted for r in res.rounds] == [3, 3, 3]
    assert [r.committed for r in res.rounds] == [4, 4, 4]
    # draft calls: prompt prefill (1 row), then per round: first call, then k-1 single rows
    per_round = draft.calls[1:]
    first_rows = [per_round[i * k][1] for i in range(3)]
    assert first_rows == [1, 2, 2]         # one behind after every fully accepted round
    # in the end the draft cache holds committed tokens only up to where it was fed
    full = [5, 6] + res.tokens
    assert draft.cache[:len(full) - 2] == full[:len(full) - 2]


def test_scripted_always_wrong_draft_is_plain_ar_speed():
    V, k = 30, 4
    tgt_t = [(t + 1) % V for t in range(V)]
    drf_t = [(t + 3) % V for t in range(V)]
    res = o.spec_generate(ScriptedLM(tgt_t, V), ScriptedLM(drf_t, V), [1], k, 9)
    assert res.tokens == [2 + i for i in range(9)]
    assert [r.accepted for r in res.rounds] == [0] * 9
    assert [r.committed for r in res.rounds] == [1] * 9


def test_scripted_eos_stops_inside_a_round():
    V, k = 30, 4
    tgt_t, drf_t = _chain(V)
    res = o.spec_generate(ScriptedLM(tgt_t, V), ScriptedLM(drf_t, V), [1, 2], k, 20, eos_id=9)
    assert res.tokens == [3, 4, 5, 6, 7, 8, 9]
    assert [r.committed for r in res.rounds] == [5, 2]
    ar = o.ar_generate(ScriptedLM(tgt_t, V), [1, 2], 20, eos_id=9)
    assert ar.tokens == res.tokens


def test_argmax_tie_goes_to_lowest_id():
    assert o.argmax_lowest(torch.tensor([0.0, 2.0, 2.0, 1.0, 2.0])) == 1


# ---------------------------------------------------------------------------
# the real tiny config: greedy speculative == autoregressive == brute force
# ---------------------------------------------------------------------------

@pytest.fixture(scope="module")
def tiny():
    w = si.make_weights(si.TINY, (1, 2))
    m = o.Model.from_shape(si.TINY, w)
    prompt = si.make_prompts(si.TINY.vocab, 1, 16)[0].tolist()
    return m, prompt


def _brute_force_greedy(m, prompt, n_new):
    y = list(prompt)
    for _ in range(n_new):
        y.append(o.argmax_lowest(o.forward_nocache(m, y)[-1]))
    return y[len(prompt):]


def test_greedy_spec_equals_ar_equals_bruteforce(tiny):
    m, prompt = tiny
    n_new = 64
    ar = o.ar_generate(o.CachedLM(m, max_seq=128), prompt, n_new).tokens
    bf = _brute_force_greedy(m, prompt, n_new)
    assert ar == bf
    for skip, k in (((1, 2), 4), ((1, 2, 3), 3), ((), 4), ((1, 2), 1), ((2,), 7)):
        kept = o.keep_layers(m.n_layers, skip)
        res = o.spec_generate(o.CachedLM(m, max_seq=128), o.CachedLM(m, kept, max_seq=128),
                              prompt, k, n_new)
        assert res.tokens == ar, (skip, k)
        assert sum(r.committed for r in res.rounds) == n_new
        for r in res.rounds[:-1]:
            assert r.committed == r.accepted + 1 and 0 <= r.accepted <= k
        if skip == ():            # draft == target: everything is accepted
            assert all(r.accepted == k for r in res.rounds)
            assert len(res.rounds) == math.ceil(n_new / (k + 1))


def test_c1_acceptance_is_meaningful(tiny):
    """Down-scaled layers {1,2} skipped: the draft agrees with the target most of the time."""
    m, prompt = tiny
    res = o.spec_generate(o.CachedLM(m, max_seq=128), o.CachedLM(m, [0, 3], max_seq=128), prompt, 4, 64)
    assert res.acceptance_rate > 0.2       # chance level is 1/2048


# ---------------------------------------------------------------------------
# sampling: exact identities
# ---------------------------------------------------------------------------

@pytest.fixture(scope="module")
def tiny64():
    w = si.make_weights(si.TINY_V64, (1, 2))
    m = o.Model.from_shape(si.TINY_V64, w)
    prompt = si.make_prompts(64, 1, 16)[0].tolist()
    return m, prompt


def test_losslessness_identity_on_real_distributions(tiny64):
    """Σ_x q(x)·min(1,p(x)/q(x))·[x=y] + P(reject)·r(y) = p(y), to fp64 rounding.
    Fails for the residual as printed in Eq. 3 (p − α_j q un-clamped) and for a
    residual that is not renormalised."""
    m, prompt = tiny64
    p = o.softmax_T(o.forward_nocache(m, prompt)[-1] * 8.0, 1.0)     # sharpened so p and q differ
    q = o.softmax_T(o.forward_nocache(m, prompt, [0, 3])[-1] * 8.0, 1.0)
    assert float((p - q).abs().max()) > 1e-3
    acc = torch.minimum(p, q)                 # q·min(1, p/q)
    beta = acc.sum()
    r = o.residual_distribution(p, q)
    out = acc + (1.0 - beta) * r
    assert float((out - p).abs().max()) < 1e-14
    assert float(r.sum()) == pytest.approx(1.0, abs=1e-14)
    assert float(r.min()) >= 0.0
    # p == q: rejection never happens and the guard returns p
    assert torch.equal(o.residual_distribution(p, p), p)


def test_softmax_temperature_literals():
    """The temperature DIVIDES the logits (reading R4; p and q of Eq. 2 are softmax(logits / T)).
    With logits (0, ln 2): T = 1 gives (1/3, 2/3); T = 1/2 doubles the gap, (1/5, 4/5); T = 2
    halves it, (1, sqrt 2) / (1 + sqrt 2).  Multiplying by T instead would swap the last two."""
    lg = torch.tensor([0.0, math.log(2.0)], dtype=torch.float32)
    assert o.softmax_T(lg, 1.0).tolist() == pytest.approx([1 / 3, 2 / 3], rel=1e-6)
    assert o.softmax_T(lg, 0.5).tolist() == pytest.approx([1 / 5, 4 / 5], rel=1e-6)
    r2 = math.sqrt(2.0)
    assert o.softmax_T(lg, 2.0).tolist() == pytest.approx([1 / (1 + r2), r2 / (1 + r2)], rel=1e-6)
    # three logits, shifted by a constant: the shift cancels, the result stays normalised
    p = o.softmax_T(torch.tensor([100.0, 100.0 + math.log(3.0), 100.0 - math.log(2.0)]), 1.0)
    assert p.tolist() == pytest.approx([1 / 4.5, 3 / 4.5, 0.5 / 4.5], rel=1e-5)
    assert float(p.sum()) == pytest.approx(1.0, abs=1e-12)


def test_categorical_inverse_cdf():
    w = torch.tensor([0.0, 2.0, 0.0, 1.0, 1.0])          # cdf: 0, .5, .5, .75, 1
    assert o.categorical(w, 0.01) == 1
    assert o.categorical(w, 0.4999) == 1
    assert o.categorical(w, 0.5001) == 3
    assert o.categorical(w, 0.76) == 4
    assert o.categorical(w, 0.999999) == 4
    # frequencies follow the weights
    cnt = np.zeros(5)
    for i in range(4000):
        cnt[o.categorical(w, philox.draw_u(3, 0, i, 0))] += 1
    assert stats.chisquare(cnt[[1, 3, 4]], np.array([.5, .25, .25]) * 4000).pvalue > 1e-3


def test_uniform01_range_and_exactness():
    assert philox.uniform01(0) == 0.5 / 2**23 > 0
    assert philox.uniform01(0xFFFFFFFF) == (2**23 - 0.5) / 2**23 < 1
    for x in (0, 1 << 9, 0x12345678, 0xFFFFFFFF):
        u = philox.uniform01(x)
        assert float(np.float32(u)) == u         # exactly representable in fp32


def test_sampling_with_draft_equal_target_accepts_everything(tiny64):
    m, prompt = tiny64
    res = o.spec_generate(o.CachedLM(m, max_seq=64), o.CachedLM(m, max_seq=64), prompt, 4, 20,
                          temperature=1.0, seed=11)
    assert all(r.accepted == 4 for r in res.rounds)


# ---------------------------------------------------------------------------
# sampling: chi-square over 1e5 seeds against exact enumeration (vocab 64)
# ---------------------------------------------------------------------------

def _merge_small(obs, exp, floor=5.0):
    """Merge cells with expectation < floor into one."""
    big = exp >= floor
    o_, e_ = list(obs[big]), list(exp[big])
    if (~big).any():
        o_.append(obs[~big].sum())
        e_.append(exp[~big].sum())
    return np.array(o_), np.array(e_)


def test_chi_square_sampled_speculative_matches_target(tiny64):
    """1e5 seeds, k=2, two new tokens each: y1 and (y1,y2) against the target's exact
    distribution.  The logits are multiplied by 8 through the temperature so that the
    distributions are far from uniform and the draft really disagrees with the target."""
    m, prompt = tiny64
    T = 1.0 / 8.0
    n_seeds = 100_000
    memo_t, memo_d = {}, {}
    kept = [0, 3]
    c1 = np.zeros(64)
    c2 = np.zeros((64, 64))
    n_rej = 0
    for seed in range(n_seeds):
        tgt, drf = o.StatelessLM(m, None, memo_t), o.StatelessLM(m, kept, memo_d)
        res = o.spec_generate(tgt, drf, prompt, 2, 2, temperature=T, seed=seed)
        c1[res.tokens[0]] += 1
        c2[res.tokens[0], res.tokens[1]] += 1
        n_rej += (res.rounds[0].accepted < 2)
    # exact target distributions by enumeration
    p1 = o.softmax_T(o.forward_nocache(m, prompt)[-1], T).numpy()
    p2 = np.stack([o.softmax_T(o.forward_nocache(m, prompt + [a])[-1], T).numpy() for a in range(64)])
    assert n_rej > 0.05 * n_seeds              # the accept/reject/residual branch is exercised
    ob, ex = _merge_small(c1, p1 * n_seeds)
    assert stats.chisquare(ob, ex).pvalue > 1e-3
    joint = p1[:, None] * p2
    ob, ex = _merge_small(c2.ravel(), joint.ravel() * n_seeds)
    assert len(ex) > 50
    assert stats.chisquare(ob, ex).pvalue > 1e-3
    # and the draft's own distribution is *not* what comes out
    q1 = o.softmax_T(o.forward_nocache(m, prompt, kept)[-1], T).numpy()
    ob, ex = _merge_small(c1, q1 * n_seeds)
    assert stats.chisquare(ob, ex * ob.sum() / ex.sum()).pvalue < 1e-6


def test_chi_square_ar_sampling(tiny64):
    m, prompt = tiny64
    T = 1.0 / 8.0
    logits = o.forward_nocache(m, prompt)[-1]
    p1 = o.softmax_T(logits, T).numpy()
    cnt = np.zeros(64)
    n = 20000
    for seed in range(n):
        cnt[o.categorical(o.softmax_T(logits, T), philox.draw_u(seed, 0, len(prompt), philox.PURPOSE_EXTRA))] += 1
    ob, ex = _merge_small(cnt, p1 * n)
    assert stats.chisquare(ob, ex).pvalue > 1e-3


def test_kv_sharing_draft_mode(tiny):
    """Reading R11.  (a) Greedy output is the target's whatever the draft reads: shared-cache
    speculative tokens == autoregressive tokens.  (b) A prune set that is a suffix of the stack
    leaves the draft's K/V equal to the target's in every layer it runs, so the shared-cache run
    reproduces the separate-cache run exactly, tokens and acceptance counts.  (c) A draft equal to
    the target accepts everything.  (d) With a prune set in the middle the two modes are
    different drafts: the acceptance counts differ somewhere."""
    m, prompt = tiny
    ar = o.ar_generate(o.CachedLM(m, max_seq=128), prompt, 40).tokens

    def run(kept, share):
        tgt = o.CachedLM(m, max_seq=128)
        drf = o.sharing_draft(tgt, kept) if share else o.CachedLM(m, kept, max_seq=128)
        return o.spec_generate(tgt, drf, prompt, 4, 40, share_kv=share)

    for kept in ([0, 3], [0, 1], [0, 1, 2, 3]):
        r = run(kept, True)
        assert r.tokens == ar
    a, b = run([0, 1], False), run([0, 1], True)
    assert [x.accepted for x in a.rounds] == [x.accepted for x in b.rounds] and a.tokens == b.tokens
    assert all(x.accepted == 4 for x in run([0, 1, 2, 3], True).rounds[:-1])
    a, b = run([0, 3], False), run([0, 3], True)
    assert [x.accepted for x in a.rounds] != [x.accepted for x in b.rounds]
