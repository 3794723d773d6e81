"""GPU parity: the CUDA library against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2602_05499_b200 as pkg
import synth_inputs as si
from oracle import sdfp_oracle as orc

from gpu_common import check_stream_against_oracle, make_pair, rel_l2

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def tiny():
    eng, m, w = make_pair(si.TINY, (1, 2))
    yield eng, m
    eng.close()


@pytest.fixture(scope="module")
def tiny_bf16():
    eng, m, w = make_pair(si.TINY_BF16, (1, 2))
    yield eng, m
    eng.close()


# ---- logits -------------------------------------------------------------------------

def _logits_both(eng, m, toks, chunks, layers=None):
    draft = layers is not None
    lm = orc.CachedLM(m, layers, max_seq=160)
    got, ref, s = [], [], 0
    for c in chunks:
        got.append(eng.sdfp_forward_logits(toks[s:s + c], s, draft=draft))
        ref.append(lm.feed(toks[s:s + c], s).numpy())
        s += c
    return np.concatenate(got), np.concatenate(ref)


def test_logits_tiny_fp32(tiny):
    eng, m = tiny
    toks = si.make_prompts(m.vocab, 1, 75, seed=5)[0].tolist()
    # ragged chunks: prefill-like 33 (three attention groups, ragged tail), single rows, a
    # verify-like 5, and a chunk crossing the 64-key attention boundary
    chunks = [33, 1, 1, 5, 20, 9, 1, 5]
    got, ref = _logits_both(eng, m, toks, chunks)
    assert got.shape == ref.shape == (75, m.vocab)
    assert rel_l2(got, ref) < 1e-4
    for r in range(75):
        assert rel_l2(got[r], ref[r]) < 1e-4, r
    got, ref = _logits_both(eng, m, toks, chunks, layers=[0, 3])
    assert rel_l2(got, ref) < 1e-4


def test_logits_tiny_bf16(tiny_bf16):
    eng, m = tiny_bf16
    toks = si.make_prompts(m.vocab, 1, 70, seed=6)[0].tolist()
    got, ref = _logits_both(eng, m, toks, [17, 1, 5, 40, 7])
    assert rel_l2(got, ref) < 1e-2
    got, ref = _logits_both(eng, m, toks, [64, 6], layers=[0, 3])
    assert rel_l2(got, ref) < 1e-2


@pytest.mark.parametrize("which", ["f32", "bf16"])
def test_rows_do_not_depend_on_batching(tiny, tiny_bf16, which):
    """Batch invariance: a row's logits are bit-identical whether its token is fed alone,
    inside a verify-sized block or inside a prefill chunk."""
    eng, m = tiny if which == "f32" else tiny_bf16
    toks = si.make_prompts(m.vocab, 1, 80, seed=8)[0].tolist()
    one = np.concatenate([eng.sdfp_forward_logits(toks[i:i + 1], i) for i in range(80)])
    s, blocks = 0, []
    for c in [5, 5, 2, 32, 1, 7, 9, 16, 3]:
        blocks.append(eng.sdfp_forward_logits(toks[s:s + c], s))
        s += c
    blk = np.concatenate(blocks)
    assert s == 80
    assert np.array_equal(one.view(np.uint32), blk.view(np.uint32))


# ---- greedy decoding ------------------------------------------------------------------

def test_greedy_c1_tokens_and_counts(tiny):
    """Config C1: 16-token prompt, 64 new tokens, skip {1,2}, k=4."""
    eng, m = tiny
    prompt = si.make_prompts(m.vocab, 1, 16)
    k, n_new = 4, 64
    out = eng.sdfp_generate(prompt, k, n_new)
    ar = eng.sdfp_generate(prompt, 0, n_new)
    assert out.tokens[0] == ar.tokens[0]                      # speculative == autoregressive on the GPU, bit-exact
    assert len(out.tokens[0]) == n_new
    reported = check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])
    ref = orc.spec_generate(orc.CachedLM(m, max_seq=160), orc.CachedLM(m, [0, 3], max_seq=160),
                            prompt[0].tolist(), k, n_new)
    if not reported:
        assert out.tokens[0] == ref.tokens
        assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]    # acceptance counts, bit-exact
        assert out.stats[:, 0, 2].tolist() == [r.committed for r in ref.rounds]
        assert out.stats[:, 0, 0].tolist() == [k] * len(ref.rounds)
        assert out.n_rounds == len(ref.rounds)
    assert ar.n_rounds == n_new and ar.stats[:, 0, 2].tolist() == [1] * n_new


@pytest.mark.parametrize("skip,k", [((1, 2, 3), 3), ((), 4), ((1, 2), 1), ((2,), 7), ((0, 1, 2), 8)])
def test_greedy_other_masks(tiny, skip, k):
    """Any draft gives the target's greedy stream; a draft equal to the target is always
    accepted; a one-layer draft is mostly rejected and exercises the rollback."""
    eng, m = tiny
    prompt = si.make_prompts(m.vocab, 1, 21, seed=77)
    n_new = 50
    eng.sdfp_set_draft_layers(si.keep_mask(4, skip))
    try:
        out = eng.sdfp_generate(prompt, k, n_new)
        ar = eng.sdfp_generate(prompt, 0, n_new)
    finally:
        eng.sdfp_set_draft_layers(si.keep_mask(4, (1, 2)))
    assert out.tokens[0] == ar.tokens[0]
    check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])
    assert int(out.stats[:, 0, 2].sum()) == n_new
    if skip == ():
        assert (out.stats[:, 0, 1] == k).all()
        assert out.n_rounds == -(-n_new // (k + 1))
    ref = orc.spec_generate(orc.CachedLM(m, max_seq=160), orc.CachedLM(m, orc.keep_layers(4, skip), max_seq=160),
                            prompt[0].tolist(), k, n_new)
    if out.tokens[0] == ref.tokens:
        assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]


@pytest.mark.parametrize("plen", [1, 2, 3, 64, 65])
def test_prompt_length_edges(tiny, plen):
    eng, m = tiny
    prompt = si.make_prompts(m.vocab, 1, plen, seed=plen)
    out = eng.sdfp_generate(prompt, 4, 12)
    ar = eng.sdfp_generate(prompt, 0, 12)
    assert out.tokens[0] == ar.tokens[0]
    check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])


def test_greedy_bf16(tiny_bf16):
    eng, m = tiny_bf16
    prompt = si.make_prompts(m.vocab, 1, 16)
    out = eng.sdfp_generate(prompt, 4, 64)
    ar = eng.sdfp_generate(prompt, 0, 64)
    assert out.tokens[0] == ar.tokens[0]
    check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])


def test_graph_and_direct_launch_agree(tiny):
    eng, m = tiny
    prompt = si.make_prompts(m.vocab, 1, 16)
    base = eng.sdfp_generate(prompt, 4, 40)
    for flags in (pkg.FLAG_NO_GRAPH, pkg.FLAG_NO_PDL, pkg.FLAG_NO_GRAPH | pkg.FLAG_NO_PDL):
        e2, _, _ = make_pair(si.TINY, (1, 2), flags=flags)
        o2 = e2.sdfp_generate(prompt, 4, 40)
        e2.close()
        assert o2.tokens == base.tokens and np.array_equal(o2.stats, base.stats)


def test_run_to_run_determinism(tiny):
    eng, m = tiny
    prompt = si.make_prompts(m.vocab, 1, 30, seed=3)
    a = eng.sdfp_generate(prompt, 4, 48)
    b = eng.sdfp_generate(prompt, 4, 48)
    assert a.tokens == b.tokens and np.array_equal(a.stats, b.stats)
    la = eng.sdfp_forward_logits(prompt[0, :20], 0)
    lb = eng.sdfp_forward_logits(prompt[0, :20], 0)
    assert np.array_equal(la.view(np.uint32), lb.view(np.uint32))


def test_eos_stops_generation():
    shape = si.TINY
    prompt = si.make_prompts(shape.vocab, 1, 16)
    eng, m, _ = make_pair(shape, (1, 2))
    full = eng.sdfp_generate(prompt, 4, 40).tokens[0]
    eng.close()
    eos = full[17]
    first = full.index(eos)
    eng, m, _ = make_pair(shape, (1, 2), eos_id=eos)
    out = eng.sdfp_generate(prompt, 4, 40)
    ar = eng.sdfp_generate(prompt, 0, 40)
    eng.close()
    assert out.tokens[0] == full[:first + 1] == ar.tokens[0]
    ref = orc.spec_generate(orc.CachedLM(m, max_seq=160), orc.CachedLM(m, [0, 3], max_seq=160),
                            prompt[0].tolist(), 4, 40, eos_id=eos)
    assert ref.tokens == out.tokens[0]
    assert out.stats[:, 0, 2].tolist() == [r.committed for r in ref.rounds]


# ---- batches ------------------------------------------------------------------------------

def test_batch_rows_are_independent():
    """A sequence's tokens and acceptance counts do not depend on what else is in the batch;
    acceptance is ragged across the batch."""
    eng, m, _ = make_pair(si.TINY, (1, 2), max_batch=4, k_max=4)
    prompts = si.make_prompts(m.vocab, 4, 24, seed=40)
    out = eng.sdfp_generate(prompts, 4, 40)
    ar = eng.sdfp_generate(prompts, 0, 40)
    assert out.tokens == ar.tokens
    for b in range(4):
        solo = eng.sdfp_generate(prompts[b:b + 1], 4, 40)
        assert solo.tokens[0] == out.tokens[b]
        acc_b = [int(a) for a, d in zip(out.stats[:, b, 1], out.stats[:, b, 0]) if d > 0]
        assert acc_b == solo.stats[:, 0, 1].tolist()
        check_stream_against_oracle(m, prompts[b].tolist(), out.tokens[b])
    eng.close()


# ---- API errors -------------------------------------------------------------------------------

def test_api_errors(tiny):
    eng, m = tiny
    prompt = si.make_prompts(m.vocab, 1, 16)
    with pytest.raises(pkg.SdfpError):
        eng.sdfp_generate(prompt, 9, 10)                    # k > k_max
    with pytest.raises(pkg.SdfpError):
        eng.sdfp_generate(prompt, 4, 200)                   # exceeds max_seq
    with pytest.raises(pkg.SdfpError):
        eng.sdfp_generate(np.full((1, 4), m.vocab, dtype=np.int32), 4, 10)   # token out of range
    with pytest.raises(pkg.SdfpError):
        eng.sdfp_generate(np.concatenate([prompt, prompt]), 4, 10)           # batch > max_batch
    with pytest.raises(pkg.SdfpError):
        eng.sdfp_set_draft_layers([0, 0, 0, 0])
    with pytest.raises(pkg.SdfpError):
        eng.sdfp_generate(prompt, 4, 10, temperature=-1.0)
    assert eng.sdfp_generate(prompt, 4, 10).tokens[0]       # still usable afterwards


# ---- 7B-shaped layers (bf16, tensor-core linear kernel at its real shapes) ----------------------

@pytest.fixture(scope="module")
def l7b4():
    eng, m, _ = make_pair(si.LLAMA7B_4L, (1, 2), max_seq=256, k_max=8, draw_device="cuda:0")
    yield eng, m
    eng.close()


def test_logits_7b_shape(l7b4):
    """d=4096, 32x128 heads, FFN 11008, vocab 32000: every linear shape of the 7B config,
    4 layers deep so that the CPU oracle finishes in seconds."""
    eng, m = l7b4
    toks = si.make_prompts(m.vocab, 1, 90, seed=9)[0].tolist()
    got, ref = _logits_both(eng, m, toks, [33, 1, 5, 2, 40, 9])
    assert rel_l2(got, ref) < 1e-2
    worst = max(rel_l2(got[r], ref[r]) for r in range(90))
    assert worst < 1e-2
    got, ref = _logits_both(eng, m, toks, [64, 1, 7], layers=[0, 3])
    assert rel_l2(got, ref) < 1e-2


def test_batch_invariance_7b_shape(l7b4):
    eng, m = l7b4
    toks = si.make_prompts(m.vocab, 1, 40, seed=10)[0].tolist()
    one = np.concatenate([eng.sdfp_forward_logits(toks[i:i + 1], i) for i in range(40)])
    s, blocks = 0, []
    for c in [5, 7, 2, 17, 9]:
        blocks.append(eng.sdfp_forward_logits(toks[s:s + c], s))
        s += c
    assert np.array_equal(one.view(np.uint32), np.concatenate(blocks).view(np.uint32))


@pytest.mark.parametrize("k", [4, 6])
def test_greedy_7b_shape(l7b4, k):
    eng, m = l7b4
    prompt = si.make_prompts(m.vocab, 1, 70, seed=12)
    out = eng.sdfp_generate(prompt, k, 48)
    ar = eng.sdfp_generate(prompt, 0, 48)
    assert out.tokens[0] == ar.tokens[0]
    reported = check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])
    assert len(reported) <= 4
    if not reported:
        ref = orc.spec_generate(orc.CachedLM(m, max_seq=256), orc.CachedLM(m, [0, 3], max_seq=256),
                                prompt[0].tolist(), k, 48)
        if ref.tokens == out.tokens[0]:
            assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]


@pytest.mark.parametrize("shape,draw", [(si.TINY_BF16, "cpu"), (si.LLAMA7B_4L, "cuda:0")])
def test_per_operation_kernels_agree_with_pass_kernel(shape, draw):
    """bf16 models run whole passes in one persistent kernel; with SDFP_FLAG_NO_PASS_KERNEL the
    same model runs one kernel per operation.  Both must match the oracle, agree closely with
    each other, and the per-operation path must keep speculative == autoregressive."""
    toks = si.make_prompts(shape.vocab, 1, 40, seed=14)[0].tolist()
    prompt = si.make_prompts(shape.vocab, 1, 20, seed=15)
    e1, m, _ = make_pair(shape, (1, 2), max_seq=128, draw_device=draw)
    a = e1.sdfp_forward_logits(toks, 0)
    g1 = e1.sdfp_generate(prompt, 4, 24)
    e1.close()
    e2, _, _ = make_pair(shape, (1, 2), max_seq=128, flags=pkg.FLAG_NO_PASS_KERNEL, draw_device=draw)
    b = e2.sdfp_forward_logits(toks, 0)
    g2 = e2.sdfp_generate(prompt, 4, 24)
    ar2 = e2.sdfp_generate(prompt, 0, 24)
    e2.close()
    ref = orc.CachedLM(m, max_seq=128).feed(toks, 0).numpy()
    assert rel_l2(a, ref) < 1e-2 and rel_l2(b, ref) < 1e-2
    assert rel_l2(a, b) < 2e-3
    assert g2.tokens == ar2.tokens
    check_stream_against_oracle(m, prompt[0].tolist(), g1.tokens[0])
    check_stream_against_oracle(m, prompt[0].tolist(), g2.tokens[0])


def test_pass_kernel_long_context_blocks(l7b4):
    """Whole-pass kernel at a context of several 64-key chunks: 16-row passes (two column groups,
    one attention item walking several chunks) give bit for bit what single-row passes give, and
    both match the oracle."""
    eng, m = l7b4
    toks = si.make_prompts(m.vocab, 1, 208, seed=16)[0].tolist()
    one = np.concatenate([eng.sdfp_forward_logits(toks[i:i + 1], i) for i in range(208)])
    blk = np.concatenate([eng.sdfp_forward_logits(toks[s:s + 16], s) for s in range(0, 208, 16)])
    assert np.array_equal(one.view(np.uint32), blk.view(np.uint32))
    five = np.concatenate([eng.sdfp_forward_logits(toks[s:s + 5], s) for s in range(100, 200, 5)])
    assert np.array_equal(one[100:200].view(np.uint32), five.view(np.uint32))
    ref = orc.CachedLM(m, max_seq=256).feed(toks, 0).numpy()
    assert max(rel_l2(blk[r], ref[r]) for r in range(208)) < 1e-2


@pytest.mark.parametrize("k", [8])
def test_greedy_wide_verify_equals_ar(tiny_bf16, l7b4, k):
    """k = 8: the verify pass carries 9 rows (two column groups) while the autoregressive pass
    carries one; the streams must still be identical."""
    for eng, m in (tiny_bf16, l7b4):
        prompt = si.make_prompts(m.vocab, 1, 70, seed=17)
        out = eng.sdfp_generate(prompt, k, 40)
        ar = eng.sdfp_generate(prompt, 0, 40)
        assert out.tokens[0] == ar.tokens[0]
        check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])


def test_time_pass_hook(l7b4):
    eng, m = l7b4
    ms, nbytes = eng.sdfp_time_pass(False, 5, 100, 4)
    d, f, v, L = 4096, 11008, 32000, 4
    want = L * (4 * d * d + 3 * d * f) * 2 + v * d * 2 + L * 2 * d * 2 * (100 + 5) + L * 2 * d * 2 * 5
    assert nbytes == want and 0.05 < ms < 50
    ms_d, nbytes_d = eng.sdfp_time_pass(True, 1, 100, 4)          # the draft keeps layers 0 and 3
    assert nbytes_d == 2 * (4 * d * d + 3 * d * f) * 2 + v * d * 2 + 2 * 2 * d * 2 * 101 + 2 * 2 * d * 2
    assert ms_d < ms


def test_13b_shape_layers():
    """d = 5120, 40 heads x 128, FFN 13824: the 13B configuration's linear and attention shapes
    (two layers deep so that the oracle finishes in seconds), logits and greedy streams."""
    shape = si.LLAMA13B_2L
    eng, m, _ = make_pair(shape, (0,), max_seq=256, k_max=8, draw_device="cuda:0")
    try:
        toks = si.make_prompts(shape.vocab, 1, 150, seed=18)[0].tolist()
        got, ref = _logits_both(eng, m, toks, [64, 33, 1, 5, 16, 31])
        assert max(rel_l2(got[r], ref[r]) for r in range(150)) < 1e-2
        prompt = si.make_prompts(shape.vocab, 1, 130, seed=19)
        out = eng.sdfp_generate(prompt, 4, 32)
        ar = eng.sdfp_generate(prompt, 0, 32)
        assert out.tokens[0] == ar.tokens[0]
        check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])
    finally:
        eng.close()


def test_batch_rows_are_independent_bf16():
    """Three sequences with k = 4 are 15 rows: they run in the whole-pass kernel as three row
    groups.  A sequence's tokens and acceptance counts must not depend on the others."""
    eng, m, _ = make_pair(si.TINY_BF16, (1, 2), max_batch=3, k_max=4)
    try:
        prompts = si.make_prompts(m.vocab, 3, 24, seed=41)
        out = eng.sdfp_generate(prompts, 4, 40)
        ar = eng.sdfp_generate(prompts, 0, 40)
        assert out.tokens == ar.tokens
        for b in range(3):
            solo = eng.sdfp_generate(prompts[b:b + 1], 4, 40)
            assert solo.tokens[0] == out.tokens[b]
            acc_b = [int(a) for a, d in zip(out.stats[:, b, 1], out.stats[:, b, 0]) if d > 0]
            assert acc_b == solo.stats[:, 0, 1].tolist()
            check_stream_against_oracle(m, prompts[b].tolist(), out.tokens[b])
    finally:
        eng.close()


def test_fma_and_tensor_paths_agree_closely():
    """The CUDA-core comparison path and the tensor-core path compute the same model."""
    shape = si.LLAMA7B_4L
    toks = si.make_prompts(shape.vocab, 1, 24, seed=13)[0].tolist()
    e1, m, _ = make_pair(shape, (1, 2), max_seq=64, draw_device="cuda:0")
    a = e1.sdfp_forward_logits(toks, 0)
    e1.close()
    e2, _, _ = make_pair(shape, (1, 2), max_seq=64, flags=pkg.FLAG_FMA_GEMM, draw_device="cuda:0")
    b = e2.sdfp_forward_logits(toks, 0)
    e2.close()
    assert rel_l2(a, b) < 2e-3


# ---- RMSNorm gains other than one ------------------------------------------------------------------

@pytest.mark.parametrize("shape,draw,tol,flags", [
    (si.TINY, "cpu", 1e-4, 0),
    (si.TINY_BF16, "cpu", 1e-2, 0),
    (si.TINY_BF16, "cpu", 1e-2, pkg.FLAG_NO_PASS_KERNEL),
    (si.TINY_BF16, "cpu", 1e-2, pkg.FLAG_FMA_GEMM),
    (si.LLAMA7B_4L, "cuda:0", 1e-2, 0),
    (si.LLAMA7B_4L, "cuda:0", 1e-2, pkg.FLAG_NO_PASS_KERNEL),
])
def test_logits_with_random_gains(shape, draw, tol, flags):
    """Every RMSNorm gain (attention norm, FFN norm, final norm of every layer) drawn from
    [0.5, 1.5): a gain applied to the wrong column, or not at all, moves the logits by tens of
    per cent.  Whole-pass kernel, per-operation tensor path and CUDA-core path."""
    eng, m, _ = make_pair(shape, (1, 2), max_seq=128, flags=flags, draw_device=draw, random_gains=True)
    try:
        toks = si.make_prompts(shape.vocab, 1, 45, seed=23)[0].tolist()
        got, ref = _logits_both(eng, m, toks, [17, 1, 5, 22])
        assert rel_l2(got, ref) < tol
        assert max(rel_l2(got[r], ref[r]) for r in range(45)) < tol
        got, ref = _logits_both(eng, m, toks, [33, 12], layers=[0, 3])
        assert rel_l2(got, ref) < tol
        # and the gains matter: the same tokens through unit gains are far away
        plain = orc.Model.from_shape(shape, si.make_weights(shape, (1, 2), device="cpu"))
        if draw == "cpu":
            far = orc.CachedLM(plain, max_seq=64).feed(toks[:8], 0).numpy()
            assert rel_l2(got[:8], far) > 0.05
    finally:
        eng.close()


# ---- one arithmetic path per context: wide contexts (batch x (k+1) > 16 rows) ----------------------

@pytest.mark.parametrize("batch,k", [(4, 4), (4, 8), (8, 2), (8, 4), (8, 8)])
def test_wide_batches_bf16(batch, k):
    """bf16 contexts whose verify pass exceeds the whole-pass kernel's 16 rows (20 .. 72 rows here)
    run every pass on the per-operation kernels.  Speculative output equals autoregressive
    output bit for bit, every sequence equals its solo run in the same context (tokens and
    acceptance counts: ragged across the batch), and every stream passes the oracle."""
    eng, m, _ = make_pair(si.TINY_BF16, (1, 2), max_seq=160, max_batch=batch, k_max=k)
    try:
        prompts = si.make_prompts(m.vocab, batch, 24, seed=50 + batch)
        n_new = 36
        out = eng.sdfp_generate(prompts, k, n_new)
        ar = eng.sdfp_generate(prompts, 0, n_new)
        assert out.tokens == ar.tokens
        ragged = set()
        for b in range(batch):
            solo = eng.sdfp_generate(prompts[b:b + 1], k, n_new)
            assert solo.tokens[0] == out.tokens[b]
            acc_b = [int(a) for a, d in zip(out.stats[:, b, 1], out.stats[:, b, 0]) if d > 0]
            assert acc_b == solo.stats[:, 0, 1].tolist()
            ragged.add(tuple(acc_b))
            check_stream_against_oracle(m, prompts[b].tolist(), out.tokens[b])
        assert len(ragged) > 1                      # the sequences really accept differently
        assert int(out.stats[:, :, 2].sum()) == batch * n_new
    finally:
        eng.close()


def test_wide_batch_7b_shape():
    """Batch 8, k = 8 (72-row verify passes, 16-row first draft passes) at the 7B layer shapes."""
    shape = si.LLAMA7B_4L
    eng, m, _ = make_pair(shape, (1, 2), max_seq=128, max_batch=8, k_max=8, draw_device="cuda:0")
    try:
        prompts = si.make_prompts(shape.vocab, 8, 40, seed=60)
        out = eng.sdfp_generate(prompts, 8, 20)
        ar = eng.sdfp_generate(prompts, 0, 20)
        assert out.tokens == ar.tokens
        for b in (0, 3, 7):
            solo = eng.sdfp_generate(prompts[b:b + 1], 8, 20)
            assert solo.tokens[0] == out.tokens[b]
            check_stream_against_oracle(m, prompts[b].tolist(), out.tokens[b])
        # rows of one forward call: the same bits whether fed one by one or 72 at a time
        toks = si.make_prompts(shape.vocab, 1, 72, seed=61)[0].tolist()
        blk = eng.sdfp_forward_logits(toks, 0)
        one = np.concatenate([eng.sdfp_forward_logits(toks[i:i + 1], i) for i in range(72)])
        assert np.array_equal(one.view(np.uint32), blk.view(np.uint32))
        ref = orc.CachedLM(m, max_seq=128).feed(toks, 0).numpy()
        assert max(rel_l2(blk[r], ref[r]) for r in range(72)) < 1e-2
    finally:
        eng.close()


def test_dense_path_long_context():
    """Decode attention of the dense path over many 64-key chunks (the ring of K/V tiles wraps, one
    split per (sequence, head) walks every chunk) and chains of linear layers behind it: contexts of
    300 to 330 keys at the 7B layer shapes, two sequences of an 8-slot context."""
    shape = si.LLAMA7B_4L
    eng, m, _ = make_pair(shape, (1, 2), max_seq=384, max_batch=8, k_max=4, draw_device="cuda:0")
    try:
        prompts = si.make_prompts(shape.vocab, 2, 300, seed=62)
        out = eng.sdfp_generate(prompts, 4, 24)
        ar = eng.sdfp_generate(prompts, 0, 24)
        assert out.tokens == ar.tokens
        assert eng.sdfp_generate(prompts[1:2], 4, 24).tokens[0] == out.tokens[1]
        check_stream_against_oracle(m, prompts[0].tolist(), out.tokens[0])
        # five rows at positions 320..324 against single rows, bit for bit, and against the oracle's logits
        toks = si.make_prompts(shape.vocab, 1, 325, seed=63)[0].tolist()
        for s0 in range(0, 320, 64):
            eng.sdfp_forward_logits(toks[s0:s0 + 64], s0)
        blk = eng.sdfp_forward_logits(toks[320:], 320)
        one = np.concatenate([eng.sdfp_forward_logits(toks[i:i + 1], i) for i in range(320, 325)])
        assert np.array_equal(one.view(np.uint32), blk.view(np.uint32))
        ref = orc.CachedLM(m, max_seq=384).feed(toks, 0).numpy()[320:]
        assert max(rel_l2(blk[r], ref[r]) for r in range(5)) < 1e-2
    finally:
        eng.close()


def test_create_accepts_72_rows_and_rejects_more():
    w = si.weights_to(si.make_weights(si.TINY_BF16, (1, 2)), "cuda:0")
    with pytest.raises(pkg.SdfpError):
        pkg.Sdfp(si.TINY_BF16, w, max_seq=64, max_batch=9, k_max=8)       # 81 rows
    eng = pkg.Sdfp(si.TINY_BF16, w, max_seq=64, max_batch=8, k_max=9)     # 80 rows
    eng.close()


# ---- the slot hand-back of the whole-pass kernel, many times over ---------------------------------

def test_pass_kernel_soak_16_rows(l7b4):
    """2000 16-row passes over the same tokens and positions: every one must give, bit for bit,
    the logits of 16 single-row passes.  (A weight slot handed back before its tile reads had
    completed once corrupted about one pass in 200 at full speed, only in wide passes.)"""
    eng, m = l7b4
    toks = si.make_prompts(m.vocab, 1, 16, seed=24)[0].tolist()
    one = np.concatenate([eng.sdfp_forward_logits(toks[i:i + 1], i) for i in range(16)]).view(np.uint32)
    bad = 0
    for it in range(2000):
        blk = eng.sdfp_forward_logits(toks, 0).view(np.uint32)
        bad += int(not np.array_equal(blk, one))
    assert bad == 0


# ---- a bounded wait that runs out --------------------------------------------------------------------

def test_wait_that_runs_out_returns_timeout(tiny_bf16):
    """Failure path of the whole-pass kernel's waits, without faulting anything: the next pass is
    told to expect one barrier arrival more than the grid has, with a 20 ms limit.  The call
    must come back quickly with SDFP_ETIMEOUT and the name of the wait, and the context must
    work again afterwards (same tokens as before)."""
    import time
    eng, m = tiny_bf16
    prompt = si.make_prompts(m.vocab, 1, 16)
    before = eng.sdfp_generate(prompt, 4, 24)
    toks = prompt[0].tolist()
    logits_before = eng.sdfp_forward_logits(toks, 0)
    eng.sdfp_debug_expire_next_wait(20_000_000)
    t0 = time.perf_counter()
    with pytest.raises(pkg.SdfpError) as ei:
        eng.sdfp_forward_logits(toks, 0)
    assert time.perf_counter() - t0 < 1.0
    assert ei.value.code == -5 and "grid barrier" in str(ei.value)
    assert np.array_equal(eng.sdfp_forward_logits(toks, 0).view(np.uint32), logits_before.view(np.uint32))
    # the same inside a generate call: the round loop stops at the first round
    eng.sdfp_debug_expire_next_wait(20_000_000)
    t0 = time.perf_counter()
    with pytest.raises(pkg.SdfpError) as ei:
        eng.sdfp_generate(prompt, 4, 24)
    assert time.perf_counter() - t0 < 1.5
    assert ei.value.code == -5
    after = eng.sdfp_generate(prompt, 4, 24)
    assert after.tokens == before.tokens and np.array_equal(after.stats, before.stats)
    ar = eng.sdfp_generate(prompt, 0, 24)
    assert ar.tokens == before.tokens


def test_dense_path_wait_that_runs_out_returns_timeout():
    """Failure path of the dense path's waits, without faulting anything: in the next forward call
    the CTAs that hold the middle of a feature tile raise their flags where nobody looks, so the CTA
    finishing the tile waits for a post that never comes, with a 20 ms limit.  The call must come back
    quickly with SDFP_ETIMEOUT and the name of the wait, the kernels behind the one that gave up must do
    nothing, and the context must work again afterwards (same logits, same tokens)."""
    import time
    eng, m, _ = make_pair(si.TINY_BF16, (1, 2), max_seq=96, max_batch=8, k_max=4)
    try:
        prompts = si.make_prompts(m.vocab, 8, 12, seed=71)
        before = eng.sdfp_generate(prompts, 4, 16)
        toks = prompts[0].tolist()
        logits_before = eng.sdfp_forward_logits(toks, 0)
        eng.sdfp_debug_expire_next_wait(20_000_000)
        t0 = time.perf_counter()
        with pytest.raises(pkg.SdfpError) as ei:
            eng.sdfp_forward_logits(toks, 0)
        assert time.perf_counter() - t0 < 1.0
        assert ei.value.code == -5 and "never posted" in str(ei.value)
        assert np.array_equal(eng.sdfp_forward_logits(toks, 0).view(np.uint32), logits_before.view(np.uint32))
        after = eng.sdfp_generate(prompts, 4, 16)   # the hook was for one forward call only
        assert after.tokens == before.tokens and np.array_equal(after.stats, before.stats)
        assert eng.sdfp_generate(prompts, 0, 16).tokens == before.tokens
    finally:
        eng.close()


# ---- the prompt pass on the tcgen05 path -------------------------------------------------------------

@pytest.mark.parametrize("shape,draw,plen", [(si.TINY_BF16, "cpu", 150), (si.TINY_BF16, "cpu", 37),
                                             (si.LLAMA7B_4L, "cuda:0", 200), (si.LLAMA13B_2L, "cuda:0", 131)])
def test_dense_prompt_pass_fills_both_caches(shape, draw, plen):
    """sdfp_generate sends the prompt through the dense kernels (tcgen05 linear layers, causal
    attention over the prompt).  What they left in the target's and in the draft's cache is read
    back through the decode kernels: the logits of the last prompt token, which attend over the
    whole cache, must match the oracle's; so must the first generated tokens; and speculative ==
    autoregressive as always.  The draft keeps layers behind the first pruned one, so both the
    copied and the recomputed part of its cache are used."""
    skip = (1,) if shape.n_layers == 2 else (1, 2)
    eng, m, _ = make_pair(shape, skip, max_seq=plen + 40, draw_device=draw)
    try:
        prompt = si.make_prompts(shape.vocab, 1, plen, seed=70)
        toks = prompt[0].tolist()
        out = eng.sdfp_generate(prompt, 4, 12)
        ar = eng.sdfp_generate(prompt, 0, 12)
        assert out.tokens == ar.tokens
        assert len(check_stream_against_oracle(m, toks, out.tokens[0])) <= 1
        eng.sdfp_generate(prompt, 4, 1)                       # caches: target 0..P-2, draft 0..P-3 from the dense pass
        ref = orc.forward_nocache(m, toks).detach().numpy()
        got = eng.sdfp_forward_logits(toks[plen - 1:], plen - 1)
        assert rel_l2(got[0], ref[plen - 1]) < 1e-2
        kept = orc.keep_layers(shape.n_layers, skip)
        ref_d = orc.forward_nocache(m, toks, kept).detach().numpy()
        got_d = eng.sdfp_forward_logits(toks[plen - 2:], plen - 2, draft=True)
        assert rel_l2(got_d[0], ref_d[plen - 2]) < 1e-2 and rel_l2(got_d[1], ref_d[plen - 1]) < 1e-2
        # the chunked prompt pass (decode kernels, SDFP_FLAG_NO_DENSE) agrees closely
        e2, _, _ = make_pair(shape, skip, max_seq=plen + 40, draw_device=draw, flags=pkg.FLAG_NO_DENSE)
        try:
            e2.sdfp_generate(prompt, 4, 1)
            alt = e2.sdfp_forward_logits(toks[plen - 1:], plen - 1)
            alt_d = e2.sdfp_forward_logits(toks[plen - 2:], plen - 2, draft=True)
        finally:
            e2.close()
        assert rel_l2(got[0], alt[0]) < 2e-3 and rel_l2(got_d, alt_d) < 2e-3
    finally:
        eng.close()


def test_dense_prompt_pass_first_layer_pruned():
    """A draft without layer 0 shares nothing with the target: its whole prompt pass is its own."""
    shape = si.TINY_BF16
    eng, m, _ = make_pair(shape, (0, 2), max_seq=160)
    try:
        prompt = si.make_prompts(shape.vocab, 1, 100, seed=71)
        toks = prompt[0].tolist()
        out = eng.sdfp_generate(prompt, 3, 10)
        assert out.tokens == eng.sdfp_generate(prompt, 0, 10).tokens
        eng.sdfp_generate(prompt, 3, 1)
        ref_d = orc.forward_nocache(m, toks, [1, 3]).detach().numpy()
        got_d = eng.sdfp_forward_logits(toks[98:], 98, draft=True)
        assert rel_l2(got_d[1], ref_d[99]) < 1e-2
    finally:
        eng.close()


def test_wide_context_without_dense_path():
    """SDFP_FLAG_NO_DENSE keeps wide contexts on the mma.sync kernels; same guarantees."""
    eng, m, _ = make_pair(si.TINY_BF16, (1, 2), max_seq=160, max_batch=4, k_max=4, flags=pkg.FLAG_NO_DENSE)
    try:
        prompts = si.make_prompts(m.vocab, 4, 24, seed=54)
        out = eng.sdfp_generate(prompts, 4, 30)
        assert out.tokens == eng.sdfp_generate(prompts, 0, 30).tokens
        for b in range(4):
            assert eng.sdfp_generate(prompts[b:b + 1], 4, 30).tokens[0] == out.tokens[b]
            check_stream_against_oracle(m, prompts[b].tolist(), out.tokens[b])
    finally:
        eng.close()


# ---- sub-layer draft masks (attention and FFN blocks pruned separately) -----------------------------

@pytest.mark.parametrize("shape,draw,flags", [(si.TINY, "cpu", 0), (si.TINY_BF16, "cpu", 0),
                                              (si.TINY_BF16, "cpu", pkg.FLAG_NO_PASS_KERNEL), (si.LLAMA7B_4L, "cuda:0", 0)])
def test_sublayer_draft_mask(shape, draw, flags):
    """The draft drops the attention block of layers 1 and 2 and the FFN block of layer 2 only
    (Section IV-A prunes the two kinds of sub-layer at different ratios).  Draft logits against
    the oracle with the same two lists; speculative == autoregressive; acceptance counts
    against the oracle's loop; a mask whose first kept block is an FFN block."""
    skip_attn, skip_ffn = (1, 2), (2,)
    pkg.build_library()
    w = si.make_weights(shape, skip_attn, device=draw, skip_ffn=skip_ffn)
    m = orc.Model.from_shape(shape, si.weights_to(w, "cpu"))
    eng = pkg.Sdfp(shape, si.weights_to(w, "cuda:0"), max_seq=200, k_max=4, flags=flags)
    try:
        ka, kf = si.keep_mask(shape.n_layers, skip_attn), si.keep_mask(shape.n_layers, skip_ffn)
        eng.sdfp_set_draft_sublayers(ka, kf)
        la, lf = orc.keep_layers(shape.n_layers, skip_attn), orc.keep_layers(shape.n_layers, skip_ffn)
        toks = si.make_prompts(shape.vocab, 1, 40, seed=80)[0].tolist()
        tol = 1e-4 if shape.dtype == "f32" else 1e-2
        lm = orc.CachedLM(m, la, max_seq=64, ffn_layers=lf)
        got = np.concatenate([eng.sdfp_forward_logits(toks[:17], 0, draft=True), eng.sdfp_forward_logits(toks[17:], 17, draft=True)])
        ref = lm.feed(toks, 0).numpy()
        assert max(rel_l2(got[r], ref[r]) for r in range(40)) < tol
        for plen in (12, 150):                       # short prompt: chunked prompt pass; long: the dense one (bf16)
            prompt = si.make_prompts(shape.vocab, 1, plen, seed=81)
            out = eng.sdfp_generate(prompt, 4, 24)
            ar = eng.sdfp_generate(prompt, 0, 24)
            assert out.tokens == ar.tokens
            rep = check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])
            ref_run = orc.spec_generate(orc.CachedLM(m, max_seq=200), orc.CachedLM(m, la, max_seq=200, ffn_layers=lf),
                                        prompt[0].tolist(), 4, 24)
            if not rep and ref_run.tokens == out.tokens[0] and shape.dtype == "f32":
                assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref_run.rounds]
        t = eng.sdfp_generate(si.make_prompts(shape.vocab, 1, 12, seed=81), 4, 24).timing
        d, f = shape.d_model, shape.d_ffn
        esz = 4 if shape.dtype == "f32" else 2
        per_draft = (len(la) * 4 * d * d + len(lf) * 3 * d * f + shape.vocab * d) * esz
        per_target = (shape.n_layers * (4 * d * d + 3 * d * f) + shape.vocab * d) * esz
        assert t["weight_bytes"] == t["n_rounds"] * (4 * per_draft + per_target)
        # a draft whose first block is an FFN block (layer 0 keeps only its FFN)
        eng.sdfp_set_draft_sublayers([0, 1, 0, 1], [1, 0, 0, 1])
        lm2 = orc.CachedLM(m, [1, 3], max_seq=64, ffn_layers=[0, 3])
        got2 = eng.sdfp_forward_logits(toks[:9], 0, draft=True)
        assert max(rel_l2(got2[r], r2) for r, r2 in enumerate(lm2.feed(toks[:9], 0).numpy())) < tol
        prompt = si.make_prompts(shape.vocab, 1, 60, seed=82)
        assert eng.sdfp_generate(prompt, 3, 16).tokens == eng.sdfp_generate(prompt, 0, 16).tokens
        with pytest.raises(pkg.SdfpError):
            eng.sdfp_set_draft_sublayers([0] * shape.n_layers, [0] * shape.n_layers)
    finally:
        eng.close()


# ---- the draft sharing the target's KV cache ---------------------------------------------------------

@pytest.mark.parametrize("which", ["f32", "bf16"])
def test_kv_sharing_draft(tiny, tiny_bf16, which):
    """sdfp_set_draft_kv_sharing: the draft attends the target's cache for the committed prefix.
    Tokens stay the target's; acceptance counts follow the oracle's loop in the same mode (fp32:
    exactly); a suffix prune set gives the same counts in both modes; switching back restores
    the separate-cache behaviour."""
    eng, m = tiny if which == "f32" else tiny_bf16
    prompt = si.make_prompts(m.vocab, 1, 90 if which == "bf16" else 16, seed=90)
    p = prompt[0].tolist()
    base = eng.sdfp_generate(prompt, 4, 40)
    ar = eng.sdfp_generate(prompt, 0, 40)
    try:
        eng.sdfp_set_draft_kv_sharing(True)
        out = eng.sdfp_generate(prompt, 4, 40)
        assert out.tokens == ar.tokens
        assert int(out.stats[:, 0, 2].sum()) == 40
        tgt = orc.CachedLM(m, max_seq=160)
        ref = orc.spec_generate(tgt, orc.sharing_draft(tgt, [0, 3]), p, 4, 40, share_kv=True)
        if which == "f32" and ref.tokens == out.tokens[0]:
            assert out.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]
        assert out.timing["kv_bytes"] < base.timing["kv_bytes"] or out.n_rounds != base.n_rounds
        # prune set = the last two layers: the shared cache holds exactly what the draft's own would
        eng.sdfp_set_draft_layers([1, 1, 0, 0])
        shared = eng.sdfp_generate(prompt, 4, 40)
        eng.sdfp_set_draft_kv_sharing(False)
        own = eng.sdfp_generate(prompt, 4, 40)
        assert shared.tokens == own.tokens == ar.tokens
        assert np.array_equal(shared.stats, own.stats)
    finally:
        eng.sdfp_set_draft_kv_sharing(False)
        eng.sdfp_set_draft_layers(si.keep_mask(4, (1, 2)))
    again = eng.sdfp_generate(prompt, 4, 40)
    assert again.tokens == base.tokens and np.array_equal(again.stats, base.stats)


def test_kv_sharing_draft_batch_and_sampling():
    """Shared cache with a batch (ragged acceptance) and with sampled decoding against the oracle."""
    eng, m, _ = make_pair(si.TINY_V64, (1, 2), max_seq=96, max_batch=3, k_max=4)
    try:
        eng.sdfp_set_draft_kv_sharing(True)
        prompts = si.make_prompts(64, 3, 20, seed=91)
        out = eng.sdfp_generate(prompts, 4, 30)
        assert out.tokens == eng.sdfp_generate(prompts, 0, 30).tokens
        for b in range(3):
            assert eng.sdfp_generate(prompts[b:b + 1], 4, 30).tokens[0] == out.tokens[b]
        same = 0
        for seed in range(12):
            g = eng.sdfp_generate(prompts[:1], 4, 20, temperature=0.125, seed=seed)
            tgt = orc.CachedLM(m, max_seq=96)
            ref = orc.spec_generate(tgt, orc.sharing_draft(tgt, [0, 3]), prompts[0].tolist(), 4, 20,
                                    temperature=0.125, seed=seed, share_kv=True)
            if g.tokens[0] == ref.tokens:
                same += 1
                assert g.stats[:, 0, 1].tolist() == [r.accepted for r in ref.rounds]
        assert same >= 11
    finally:
        eng.close()


def test_dense_path_sublayer_mask_and_kv_sharing():
    """The two draft variants on a context whose passes run on the dense path (8 sequence slots):
    a sub-layer mask whose draft stack has an attention-only and an FFN-only layer (draft logits
    against the oracle with the same two lists), and the draft attending the target's cache.
    Tokens stay the target's in a batch with ragged acceptance; each sequence equals its solo run."""
    shape = si.TINY_BF16
    skip_attn, skip_ffn = (1, 2), (2,)
    pkg.build_library()
    w = si.make_weights(shape, skip_attn, skip_ffn=skip_ffn)
    m = orc.Model.from_shape(shape, si.weights_to(w, "cpu"))
    eng = pkg.Sdfp(shape, si.weights_to(w, "cuda:0"), max_seq=128, max_batch=8, k_max=4)
    try:
        ka, kf = si.keep_mask(shape.n_layers, skip_attn), si.keep_mask(shape.n_layers, skip_ffn)
        eng.sdfp_set_draft_sublayers(ka, kf)
        la, lf = orc.keep_layers(shape.n_layers, skip_attn), orc.keep_layers(shape.n_layers, skip_ffn)
        toks = si.make_prompts(shape.vocab, 1, 40, seed=84)[0].tolist()
        got = np.concatenate([eng.sdfp_forward_logits(toks[:17], 0, draft=True), eng.sdfp_forward_logits(toks[17:], 17, draft=True)])
        ref = orc.CachedLM(m, la, max_seq=64, ffn_layers=lf).feed(toks, 0).numpy()
        assert max(rel_l2(got[r], ref[r]) for r in range(40)) < 1e-2
        prompts = si.make_prompts(shape.vocab, 8, 30, seed=85)
        ar = eng.sdfp_generate(prompts, 0, 24)
        for share in (False, True):
            eng.sdfp_set_draft_kv_sharing(share)
            out = eng.sdfp_generate(prompts, 4, 24)
            assert out.tokens == ar.tokens
            assert len({int(x) for x in out.stats[:, :, 1].ravel()}) > 1      # acceptance is ragged
            for b in (0, 5):
                assert eng.sdfp_generate(prompts[b:b + 1], 4, 24).tokens[0] == out.tokens[b]
        check_stream_against_oracle(m, prompts[3].tolist(), ar.tokens[3])
    finally:
        eng.sdfp_set_draft_kv_sharing(False)
        eng.close()


def test_bf16_error_budget_against_unrounded_cache(tiny_bf16, l7b4, capsys):
    """The bf16 configurations round K/V to bf16 on both sides (oracle and library).  Against an
    oracle that keeps K/V in fp32 the library's logits must still sit inside the same tolerance;
    both figures are printed (run with -s) so that the share of the K/V rounding is on record."""
    import dataclasses
    for name, (eng, m) in (("tiny-bf16", tiny_bf16), ("7b-4layers", l7b4)):
        toks = si.make_prompts(m.vocab, 1, 100, seed=95)[0].tolist()
        got = np.concatenate([eng.sdfp_forward_logits(toks[:64], 0), eng.sdfp_forward_logits(toks[64:], 64)])
        same = orc.forward_nocache(m, toks).detach().numpy()
        unrounded = orc.forward_nocache(dataclasses.replace(m, kv_bf16=False), toks).detach().numpy()
        e_same, e_unr, e_kv = rel_l2(got, same), rel_l2(got, unrounded), rel_l2(same, unrounded)
        with capsys.disabled():
            print("\n[bf16 error budget] %s: library vs oracle (K/V rounded on both sides) %.3e; library vs oracle with fp32 K/V %.3e; "
                  "the two oracles against each other %.3e" % (name, e_same, e_unr, e_kv))
        assert e_same < 1e-2 and e_unr < 1e-2


def test_long_context_against_oracle():
    """The 13B configuration's context length (2048-token prompt, keys up to ~2300) at the 7B layer
    shapes, four layers deep: the prompt goes through the dense path in 16 row blocks, decode
    attention walks 33+ chunks of 64 keys per head (4-5 per split), and every generated token is
    checked against the oracle's recomputation of the whole sequence."""
    shape = si.LLAMA7B_4L
    plen, n_new = 2048, 40
    eng, m, _ = make_pair(shape, (1, 2), max_seq=plen + n_new + 16, k_max=4, draw_device="cuda:0")
    try:
        prompt = si.make_prompts(shape.vocab, 1, plen, seed=96)
        out = eng.sdfp_generate(prompt, 4, n_new)
        ar = eng.sdfp_generate(prompt, 0, n_new)
        assert out.tokens == ar.tokens
        reported = check_stream_against_oracle(m, prompt[0].tolist(), out.tokens[0])
        assert len(reported) <= 2, reported
        # logits of three more positions through the decode kernels over the 2088-key cache
        toks = prompt[0].tolist() + out.tokens[0]
        got = eng.sdfp_forward_logits(toks[-3:], len(toks) - 3)
        ref = orc.forward_nocache(m, toks).detach().numpy()[-3:]
        assert max(rel_l2(got[r], ref[r]) for r in range(3)) < 1e-2
    finally:
        eng.close()


def test_time_linear_hook_on_both_bf16_paths():
    """The roofline hook of the linear kernels: per-operation mma.sync kernels (flag) and the tcgen05
    kernel of a wide context; bytes are the matrix's, times are sane."""
    shape = si.LLAMA7B_4L
    d, f, v = shape.d_model, shape.d_ffn, shape.vocab
    want = [3 * d * d * 2, d * d * 2, 2 * f * d * 2, d * f * 2, v * d * 2]
    for kw in (dict(flags=pkg.FLAG_NO_PASS_KERNEL), dict(max_batch=8, k_max=4)):
        eng, _, _ = make_pair(shape, (1, 2), max_seq=128, draw_device="cuda:0", **kw)
        try:
            for which in range(5):
                ms, nbytes = eng.sdfp_time_linear(which, 8, 8)
                assert nbytes == want[which] and 0.002 < ms < 5.0
            with pytest.raises(pkg.SdfpError):
                eng.sdfp_time_pass(False, 1, 0, 2)            # neither context runs the whole-pass kernel
        finally:
            eng.close()


def test_largest_batch_and_row_count():
    """The library's limits in one context: 16 sequences, k = 4, 80 rows in a verify pass (row block of
    80 rows = MMA width 160), 32 rows in the first draft pass; prompts of one token (nothing to cache
    before the first round).  Speculative == autoregressive, sequences independent."""
    eng, m, _ = make_pair(si.TINY_BF16, (1, 2), max_seq=64, max_batch=16, k_max=4)
    try:
        for plen in (1, 9):
            prompts = si.make_prompts(m.vocab, 16, plen, seed=97)
            out = eng.sdfp_generate(prompts, 4, 20)
            assert out.tokens == eng.sdfp_generate(prompts, 0, 20).tokens
            for b in (0, 7, 15):
                assert eng.sdfp_generate(prompts[b:b + 1], 4, 20).tokens[0] == out.tokens[b]
                check_stream_against_oracle(m, prompts[b].tolist(), out.tokens[b])
    finally:
        eng.close()
