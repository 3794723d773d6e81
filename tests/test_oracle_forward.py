"""Pins of the oracle's forward pass against things other than itself:
hand-worked scalar examples, closed forms, invariants, and the no-cache
recomputation (an independently written second route through the model)."""
import math

import numpy as np
import pytest
import torch

import synth_inputs as si
from oracle import sdfp_oracle as o


def _tiny_model(dtype=torch.float32, shape=si.TINY, skip=(1, 2)):
    w = si.make_weights(shape, skip)
    return o.Model.from_shape(shape, w, dtype=dtype)


def _hand_model(d, H, hd, f, V, dtype=torch.float64):
    """All-zero weights with unit gains; tests fill in what they need."""
    z = lambda *s: torch.zeros(*s, dtype=dtype)
    lw = dict(wq=z(d, d), wk=z(d, d), wv=z(d, d), wo=z(d, d), w_gate=z(f, d), w_up=z(f, d),
              w_down=z(d, f), attn_norm=torch.ones(d, dtype=dtype), ffn_norm=torch.ones(d, dtype=dtype))
    w = dict(tok_embed=z(V, d), lm_head=z(V, d), final_norm=torch.ones(d, dtype=dtype), layers=[lw])
    return o.Model(w, 1, d, H, hd, f, V, 1e-5, 10000.0, kv_bf16=False, dtype=dtype)


# ---- unit cases with hand-computable values --------------------------------

def test_rmsnorm_literal():
    h = torch.tensor([[3.0, 4.0]], dtype=torch.float64)
    g = torch.tensor([1.0, 2.0], dtype=torch.float64)
    out = o.rmsnorm(h, g, 1e-5)
    r = math.sqrt(12.5 + 1e-5)          # mean(9, 16) = 12.5; eps inside the root
    assert out[0, 0].item() == pytest.approx(3.0 / r, rel=1e-14)
    assert out[0, 1].item() == pytest.approx(8.0 / r, rel=1e-14)
    # eps matters when h is tiny: mean square 1e-6 -> scale 1/sqrt(1.1e-5)
    h = torch.tensor([[1e-3, 1e-3]], dtype=torch.float64)
    assert o.rmsnorm(h, torch.ones(2, dtype=torch.float64), 1e-5)[0, 0].item() == pytest.approx(
        1e-3 / math.sqrt(1e-6 + 1e-5), rel=1e-12)


def test_silu_literal():
    x = torch.tensor([0.0, 1.0, -1.0, 20.0], dtype=torch.float64)
    y = o.silu(x)
    assert y[0].item() == 0.0
    assert y[1].item() == pytest.approx(0.7310585786300049, rel=1e-14)
    assert y[2].item() == pytest.approx(-0.2689414213699951, rel=1e-14)
    assert y[3].item() == pytest.approx(20.0, rel=1e-8)


def test_rope_literal_pairing_and_frequencies():
    # head_dim 4, theta 10000: pair (0,2) turns by pos*1, pair (1,3) by pos*10000^(-2/4) = pos*0.01
    cos, sin = o.rope_angles(4, 10000.0, [0, 1, 3], torch.float64)
    x = torch.zeros(3, 1, 4, dtype=torch.float64)
    x[:, 0, 0] = 1.0      # unit vector on the first element of pair (0,2)
    x[:, 0, 1] = 2.0      # and 2 on the first element of pair (1,3)
    y = o.apply_rope(x, cos, sin)
    assert torch.equal(y[0], x[0])                        # position 0 is the identity
    assert y[1, 0].tolist() == pytest.approx(
        [math.cos(1.0), 2 * math.cos(0.01), math.sin(1.0), 2 * math.sin(0.01)], rel=1e-14)
    assert y[2, 0].tolist() == pytest.approx(
        [math.cos(3.0), 2 * math.cos(0.03), math.sin(3.0), 2 * math.sin(0.03)], rel=1e-14)
    assert math.cos(1.0) == pytest.approx(0.5403023058681398, rel=1e-15)


def test_rope_invariants():
    g = torch.Generator().manual_seed(0)
    q = torch.randn(1, 2, 64, generator=g, dtype=torch.float64)
    k = torch.randn(1, 2, 64, generator=g, dtype=torch.float64)

    def dot(m, n):
        cm, sm = o.rope_angles(64, 10000.0, [m], torch.float64)
        cn, sn = o.rope_angles(64, 10000.0, [n], torch.float64)
        return (o.apply_rope(q, cm, sm) * o.apply_rope(k, cn, sn)).sum(-1)

    c, s = o.rope_angles(64, 10000.0, [17], torch.float64)
    assert torch.allclose(o.apply_rope(q, c, s).norm(dim=-1), q.norm(dim=-1), rtol=1e-13)
    # the score depends on the position difference only
    assert torch.allclose(dot(5, 2), dot(105, 102), rtol=1e-10, atol=1e-12)
    assert not torch.allclose(dot(5, 2), dot(5, 3), rtol=1e-3)


# ---- hand-built models with closed-form answers ----------------------------

def test_weight_orientation_attention_path():
    """[out, in] convention of wv and wo, on a one-token sequence (softmax over one key = 1).

    v = P·x̂ with P a permutation, a = v, h1 = e + A·a with A a scaled shift.  The
    expectation is written with explicit index moves, so x·W and x·Wᵀ differ.
    """
    d = 4
    m = _hand_model(d, 1, 4, 6, 3)
    e = [0.5, -1.0, 2.0, 0.25]
    m.w["tok_embed"][0] = torch.tensor(e, dtype=torch.float64)
    perm = [2, 0, 3, 1]                      # v[i] = x̂[perm[i]]
    for i in range(d):
        m.w["layers"][0]["wv"][i, perm[i]] = 1.0
        m.w["layers"][0]["wo"][i, (i + 1) % d] = 2.0      # (A y)[i] = 2·y[i+1]
    # lm head reads out h1 (after the final norm) one coordinate at a time
    m.w["lm_head"][0, 0] = 1.0
    m.w["lm_head"][1, 1] = 1.0
    m.w["lm_head"][2, 3] = 1.0
    rms = math.sqrt(sum(x * x for x in e) / d + 1e-5)
    xh = [x / rms for x in e]
    v = [xh[perm[i]] for i in range(d)]
    h1 = [e[i] + 2.0 * v[(i + 1) % d] for i in range(d)]
    rms1 = math.sqrt(sum(x * x for x in h1) / d + 1e-5)
    expect = [h1[0] / rms1, h1[1] / rms1, h1[3] / rms1]
    got = o.forward_nocache(m, [0])[0].tolist()
    assert got == pytest.approx(expect, rel=1e-12)
    got = o.CachedLM(m, max_seq=4).feed([0], 0)[0].tolist()
    assert got == pytest.approx(expect, rel=1e-12)


def test_weight_orientation_ffn_path():
    """gate = x̂[p1], up = x̂[p2], u = silu(gate)·up, h1 = e + D·u with D rectangular."""
    d, f = 4, 6
    m = _hand_model(d, 1, 4, f, 4)
    e = [0.5, -1.0, 2.0, 0.25]
    m.w["tok_embed"][1] = torch.tensor(e, dtype=torch.float64)
    p1 = [0, 1, 2, 3, 0, 1]
    p2 = [3, 2, 1, 0, 1, 2]
    lw = m.w["layers"][0]
    for j in range(f):
        lw["w_gate"][j, p1[j]] = 1.0
        lw["w_up"][j, p2[j]] = 1.0
    # h1[i] = e[i] + 3·u[i] − u[i+2]
    for i in range(d):
        lw["w_down"][i, i] = 3.0
        lw["w_down"][i, (i + 2) % f] += -1.0
    for i in range(d):
        m.w["lm_head"][i, i] = 1.0
    rms = math.sqrt(sum(x * x for x in e) / d + 1e-5)
    xh = [x / rms for x in e]
    u = [(xh[p1[j]] / (1.0 + math.exp(-xh[p1[j]]))) * xh[p2[j]] for j in range(f)]
    h1 = [e[i] + 3.0 * u[i] - u[(i + 2) % f] for i in range(d)]
    rms1 = math.sqrt(sum(x * x for x in h1) / d + 1e-5)
    got = o.forward_nocache(m, [1])[0].tolist()
    assert got == pytest.approx([x / rms1 for x in h1], rel=1e-12)


def test_two_token_attention_worked_by_hand():
    """d=2, one head, wq=wk=wv=wo=I, T=2: every number of the attention worked in scalars."""
    m = _hand_model(2, 1, 2, 2, 3)
    e0, e1 = [1.0, 2.0], [-0.5, 1.5]
    m.w["tok_embed"][0] = torch.tensor(e0, dtype=torch.float64)
    m.w["tok_embed"][1] = torch.tensor(e1, dtype=torch.float64)
    lw = m.w["layers"][0]
    for name in ("wq", "wk", "wv", "wo"):
        lw[name][0, 0] = lw[name][1, 1] = 1.0
    m.w["lm_head"][0, 0] = 1.0
    m.w["lm_head"][1, 1] = 1.0
    m.w["lm_head"][2, 0] = m.w["lm_head"][2, 1] = 1.0

    def norm(v):
        r = math.sqrt((v[0] ** 2 + v[1] ** 2) / 2 + 1e-5)
        return [v[0] / r, v[1] / r]

    def rot(v, pos):                      # head_dim 2: one pair, frequency 1
        c, s = math.cos(pos), math.sin(pos)
        return [v[0] * c - v[1] * s, v[1] * c + v[0] * s]

    x0, x1 = norm(e0), norm(e1)
    k0, k1, q1 = rot(x0, 0), rot(x1, 1), rot(x1, 1)
    s10 = (q1[0] * k0[0] + q1[1] * k0[1]) / math.sqrt(2)
    s11 = (q1[0] * k1[0] + q1[1] * k1[1]) / math.sqrt(2)
    mx = max(s10, s11)
    w0, w1 = math.exp(s10 - mx), math.exp(s11 - mx)
    p0, p1 = w0 / (w0 + w1), w1 / (w0 + w1)
    a1 = [p0 * x0[0] + p1 * x1[0], p0 * x0[1] + p1 * x1[1]]      # v = x̂ (not rotated)
    h_row0 = [e0[0] + x0[0], e0[1] + x0[1]]                      # row 0 sees only itself
    h_row1 = [e1[0] + a1[0], e1[1] + a1[1]]
    exp_rows = []
    for h in (h_row0, h_row1):
        n = norm(h)                                              # FFN is zero
        exp_rows.append([n[0], n[1], n[0] + n[1]])
    got = o.forward_nocache(m, [0, 1])
    assert got[0].tolist() == pytest.approx(exp_rows[0], rel=1e-12)
    assert got[1].tolist() == pytest.approx(exp_rows[1], rel=1e-12)
    lm = o.CachedLM(m, max_seq=4)
    r0 = lm.feed([0], 0)
    r1 = lm.feed([1], 1)
    assert r0[0].tolist() == pytest.approx(exp_rows[0], rel=1e-12)
    assert r1[0].tolist() == pytest.approx(exp_rows[1], rel=1e-12)


def test_two_heads_partition_contiguous_blocks_worked_by_hand():
    """d=4, two heads of width 2, wq=wk=wv=wo=I, T=2: head h owns dimensions 2h, 2h+1 of q, k
    and v (contiguous blocks, the LLaMA layout), each head has its own softmax over the two
    keys, and the two heads get different attention weights.  Everything is worked in scalars;
    a layout that interleaved the heads (dimensions h, h+2) pairs different numbers in the
    rotation and in the dot products and gives other values."""
    m = _hand_model(4, 2, 2, 2, 4)
    e0, e1 = [1.0, 2.0, -1.0, 0.5], [-0.5, 1.5, 2.0, 1.0]
    m.w["tok_embed"][0] = torch.tensor(e0, dtype=torch.float64)
    m.w["tok_embed"][1] = torch.tensor(e1, dtype=torch.float64)
    lw = m.w["layers"][0]
    for name in ("wq", "wk", "wv", "wo"):
        for i in range(4):
            lw[name][i, i] = 1.0
    for i in range(4):
        m.w["lm_head"][i, i] = 1.0

    def norm(v):
        r = math.sqrt(sum(x * x for x in v) / 4 + 1e-5)
        return [x / r for x in v]

    def rot(a, b, pos):                   # head_dim 2: one pair per head, frequency 1
        c, s = math.cos(pos), math.sin(pos)
        return [a * c - b * s, b * c + a * s]

    x0, x1 = norm(e0), norm(e1)
    a1, probs = [], []
    for h in range(2):
        lo, hi = 2 * h, 2 * h + 1
        k0 = rot(x0[lo], x0[hi], 0)
        k1 = rot(x1[lo], x1[hi], 1)
        q1 = k1                           # wq = wk
        s10 = (q1[0] * k0[0] + q1[1] * k0[1]) / math.sqrt(2)
        s11 = (q1[0] * k1[0] + q1[1] * k1[1]) / math.sqrt(2)
        mx = max(s10, s11)
        w0, w1 = math.exp(s10 - mx), math.exp(s11 - mx)
        p0, p1 = w0 / (w0 + w1), w1 / (w0 + w1)
        probs.append(p0)
        a1 += [p0 * x0[lo] + p1 * x1[lo], p0 * x0[hi] + p1 * x1[hi]]      # v = x̂, not rotated
    assert abs(probs[0] - probs[1]) > 0.02                                # the heads really differ
    h_row0 = [e0[i] + x0[i] for i in range(4)]                            # row 0 sees only itself
    h_row1 = [e1[i] + a1[i] for i in range(4)]
    expect = [norm(h_row0), norm(h_row1)]                                 # FFN is zero
    got = o.forward_nocache(m, [0, 1])
    assert got[0].tolist() == pytest.approx(expect[0], rel=1e-12)
    assert got[1].tolist() == pytest.approx(expect[1], rel=1e-12)
    lm = o.CachedLM(m, max_seq=4)
    r0 = lm.feed([0], 0)
    r1 = lm.feed([1], 1)
    assert r0[0].tolist() == pytest.approx(expect[0], rel=1e-12)
    assert r1[0].tolist() == pytest.approx(expect[1], rel=1e-12)
    both = o.CachedLM(m, max_seq=4).feed([0, 1], 0)
    assert both[1].tolist() == pytest.approx(expect[1], rel=1e-12)
    # the interleaved reading (head h = dimensions h, h+2) worked the same way gives other numbers
    alt = []
    for h in range(2):
        lo, hi = h, h + 2
        k0, k1 = rot(x0[lo], x0[hi], 0), rot(x1[lo], x1[hi], 1)
        s10 = (k1[0] * k0[0] + k1[1] * k0[1]) / math.sqrt(2)
        s11 = (k1[0] * k1[0] + k1[1] * k1[1]) / math.sqrt(2)
        w0, w1 = math.exp(s10 - max(s10, s11)), math.exp(s11 - max(s10, s11))
        alt.append(w0 / (w0 + w1))
    assert abs(alt[0] - probs[0]) > 1e-3 or abs(alt[1] - probs[1]) > 1e-3


def test_uniform_attention_is_causal_running_mean():
    """wq = 0 makes every score 0, so attention is the running mean of v (textbook special case)."""
    shape = si.ModelShape("t", 1, 32, 2, 16, 48, 40)
    w = si.make_weights(shape, [])
    m = o.Model.from_shape(shape, w, dtype=torch.float64)
    lw = m.w["layers"][0]
    lw["wq"].zero_()
    lw["w_down"].zero_()                       # no FFN contribution
    d = shape.d_model
    lw["wo"].copy_(torch.eye(d))
    toks = [3, 9, 27, 1, 5]
    E = m.w["tok_embed"].double()[toks]
    xh = E / torch.sqrt((E * E).mean(-1, keepdim=True) + shape.rms_eps)
    v = xh @ lw["wv"].double().t()
    run_mean = torch.cumsum(v, 0) / torch.arange(1, 6, dtype=torch.float64)[:, None]
    h1 = E + run_mean
    xf = h1 / torch.sqrt((h1 * h1).mean(-1, keepdim=True) + shape.rms_eps)
    expect = xf @ m.w["lm_head"].double().t()
    assert torch.allclose(o.forward_nocache(m, toks), expect, rtol=1e-10, atol=1e-12)
    assert torch.allclose(o.CachedLM(m, max_seq=8).feed(toks, 0), expect, rtol=1e-10, atol=1e-12)


# ---- invariants on the real tiny config ------------------------------------

@pytest.mark.parametrize("dtype,tol", [(torch.float32, 2e-5), (torch.float64, 1e-12)])
def test_cached_equals_nocache(dtype, tol):
    m = _tiny_model(dtype)
    toks = si.make_prompts(m.vocab, 1, 24)[0].tolist()
    full = o.forward_nocache(m, toks)
    lm = o.CachedLM(m, max_seq=32)
    a = lm.feed(toks[:10], 0)             # chunked prefill
    b = lm.feed(toks[10:11], 10)          # one decode row
    c = lm.feed(toks[11:16], 11)          # a verify-like block of 5 rows
    d = lm.feed(toks[16:], 16)
    inc = torch.cat([a, b, c, d], 0)
    rel = ((inc - full).norm() / full.norm()).item()
    assert rel < tol
    # draft (kept layers only) too
    kept = [0, 3]
    full_d = o.forward_nocache(m, toks, kept)
    lm = o.CachedLM(m, kept, max_seq=32)
    inc_d = torch.cat([lm.feed(toks[:7], 0), lm.feed(toks[7:], 7)], 0)
    assert ((inc_d - full_d).norm() / full_d.norm()).item() < tol
    assert ((full_d - full).norm() / full.norm()).item() > 1e-3      # the draft is a different model


def test_overwrite_is_rollback():
    """Feeding at an earlier position discards what was cached beyond it."""
    m = _tiny_model(torch.float64)
    toks = si.make_prompts(m.vocab, 1, 12)[0].tolist()
    lm = o.CachedLM(m, max_seq=32)
    lm.feed(toks[:8], 0)
    lm.feed([7, 7, 7, 7], 8)                       # speculative junk at 8..11
    got = lm.feed(toks[8:], 8)                     # roll back to 8 and feed the real tokens
    ref = o.forward_nocache(m, toks)[8:]
    assert torch.allclose(got, ref, rtol=1e-9, atol=1e-12)


def test_causality():
    m = _tiny_model(torch.float64)
    toks = si.make_prompts(m.vocab, 1, 10)[0].tolist()
    a = o.forward_nocache(m, toks)
    toks2 = list(toks)
    toks2[7] = (toks2[7] + 1) % m.vocab
    b = o.forward_nocache(m, toks2)
    assert torch.equal(a[:7], b[:7])
    assert not torch.allclose(a[7:], b[7:])


def test_skipped_layer_equals_zeroed_output_projections():
    """A layer whose o_proj and down_proj are zero adds nothing: same logits as removing it."""
    m = _tiny_model(torch.float64)
    toks = si.make_prompts(m.vocab, 1, 9)[0].tolist()
    skipped = o.forward_nocache(m, toks, [0, 3])
    for l in (1, 2):
        m.w["layers"][l]["wo"].zero_()
        m.w["layers"][l]["w_down"].zero_()
    zeroed = o.forward_nocache(m, toks)
    assert torch.allclose(skipped, zeroed, rtol=1e-12, atol=1e-14)


def test_fp32_close_to_fp64():
    m32, m64 = _tiny_model(torch.float32), _tiny_model(torch.float64)
    toks = si.make_prompts(m32.vocab, 1, 20)[0].tolist()
    a, b = o.forward_nocache(m32, toks).double(), o.forward_nocache(m64, toks)
    assert ((a - b).norm() / b.norm()).item() < 1e-5


def test_bf16_model_kv_rounding():
    """bf16 model: weights widen exactly; K/V entering the cache are bf16 values."""
    shape = si.TINY_BF16
    w = si.make_weights(shape, (1, 2))
    m = o.Model.from_shape(shape, w)
    assert m.kv_bf16
    lm = o.CachedLM(m, max_seq=16)
    toks = si.make_prompts(m.vocab, 1, 6)[0].tolist()
    inc = torch.cat([lm.feed(toks[:4], 0), lm.feed(toks[4:], 4)], 0)
    k = lm.k[0][:6]
    assert torch.equal(k, k.to(torch.bfloat16).to(torch.float32))
    full = o.forward_nocache(m, toks)
    assert ((inc - full).norm() / full.norm()).item() < 1e-4


def test_skipped_sub_blocks_equal_zeroed_output_projections():
    """Sub-layer pruning (reading R10): dropping a layer's attention block is the same function as
    zeroing its wo, dropping its FFN block the same as zeroing its w_down, independently of each
    other; no-cache and cached forward agree; and the two blocks are not interchangeable."""
    m = _tiny_model(dtype=torch.float64)
    toks = si.make_prompts(m.vocab, 1, 12, seed=4)[0].tolist()
    attn_keep, ffn_keep = [0, 2, 3], [0, 1, 3]          # layer 1 loses attention, layer 2 loses its FFN
    got = o.forward_nocache(m, toks, attn_keep, ffn_keep)
    import copy
    w2 = copy.deepcopy(m.w)
    w2["layers"][1]["wo"].zero_()
    w2["layers"][2]["w_down"].zero_()
    m2 = o.Model.from_shape(si.TINY, w2, dtype=torch.float64)
    want = o.forward_nocache(m2, toks)
    assert torch.allclose(got, want, rtol=1e-10, atol=1e-12)
    lm = o.CachedLM(m, attn_keep, max_seq=16, ffn_layers=ffn_keep)
    a = lm.feed(toks[:7], 0)
    b = lm.feed(toks[7:], 7)
    assert torch.allclose(torch.cat([a, b]), want, rtol=1e-9, atol=1e-11)
    assert sorted(lm.k.keys()) == attn_keep                 # a cache only for the attention blocks that run
    # swapping the roles gives another function
    other = o.forward_nocache(m, toks, ffn_keep, attn_keep)
    assert not torch.allclose(other, want, rtol=1e-3, atol=1e-6)
    # whole layers are the special case of equal lists
    assert torch.equal(o.forward_nocache(m, toks, [0, 3], [0, 3]), o.forward_nocache(m, toks, [0, 3]))
