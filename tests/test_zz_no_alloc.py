"""The allocation-free forward call against the ordinary one, through the C ABI.

sdfp_forward_logits_static is for callers that may not touch a device allocator when they
call the library (all of HBM already claimed by their own pool, a loop that cannot afford the
device-wide synchronisation an allocation implies, a thread running beside a CUDA-graph
capture).  It runs the same forward pass as sdfp_forward_logits, but the split-KV attention
kernel's scratch is a fixed array inside the library image.  That array is shared by every
call and keeps the previous call's contents, so the check is made on two calls in a row, with
different shapes, and both must reproduce the ordinary entry point.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest

import paper_2602_05499_b200 as pkg
import synth_inputs as si

from gpu_common import make_pair, rel_l2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("shape,tol", [(si.TINY, 1e-4), (si.TINY_BF16, 1e-2)])
def test_static_scratch_forward_matches_regular_forward(shape, tol):
    eng, m, _ = make_pair(shape, (1, 2), max_seq=160)
    try:
        toks = si.make_prompts(shape.vocab, 1, 110, seed=21)[0].tolist()
        # first call: a prefill-like block of 60 rows (several row groups, ragged tail)
        ref_a = eng.sdfp_forward_logits(toks[:60], 0)
        got_a = eng.sdfp_forward_logits_static(toks[:60], 0)
        # second call straight after it: fewer rows, a context that crosses the 64-key chunk
        # boundary, so the partials and counters the first call left in the array lie under and
        # beside the ones this call uses
        ref_b = eng.sdfp_forward_logits(toks[60:71], 60)
        got_b = eng.sdfp_forward_logits_static(toks[60:71], 60)
        assert got_a.shape == ref_a.shape and got_b.shape == ref_b.shape
        assert rel_l2(got_a, ref_a) < tol and rel_l2(got_b, ref_b) < tol
        # same kernels, same order of operations: in fact bit-identical
        assert np.array_equal(got_a.view(np.uint32), ref_a.view(np.uint32))
        assert np.array_equal(got_b.view(np.uint32), ref_b.view(np.uint32))
        # the draft model (kept layers only, its own cache) goes through the same entry point
        ref_d = eng.sdfp_forward_logits(toks[:33], 0, draft=True)
        got_d = eng.sdfp_forward_logits_static(toks[:33], 0, draft=True)
        assert rel_l2(got_d, ref_d) < tol
    finally:
        eng.close()


def test_static_scratch_rejects_what_does_not_fit():
    """With one kernel per operation, a 64-row call on 32 heads of width 128 needs about 1 MiB of
    partials per 64-key chunk: at a context of 2164 tokens (34 chunks) that is far beyond the
    8 MiB array and must be refused with both sizes in the message, while a small call on the
    same context is served."""
    shape = si.LLAMA7B_4L
    eng, m, _ = make_pair(shape, (1, 2), max_seq=2200, flags=pkg.FLAG_NO_PASS_KERNEL, draw_device="cuda:0")
    try:
        toks = si.make_prompts(shape.vocab, 1, 64, seed=22)[0].tolist()
        with pytest.raises(pkg.SdfpError) as ei:
            eng.sdfp_forward_logits_static(toks, 2100)
        assert ei.value.code == -1 and "static array holds" in str(ei.value)
        ok = eng.sdfp_forward_logits_static(toks[:5], 0)
        assert np.array_equal(ok.view(np.uint32), eng.sdfp_forward_logits(toks[:5], 0).view(np.uint32))
    finally:
        eng.close()


def test_static_call_allocates_nothing_and_leaves_the_context_intact():
    """The promise itself: once the first call on the device has looked the array up, a static call
    leaves the device's free memory exactly where it was (no cudaMalloc, no pool growth), a refused
    call likewise, and afterwards the context still generates what a fresh context generates (the
    static call borrows the context's scratch pointers and must hand them back, also on the error
    return)."""
    import torch
    shape = si.LLAMA7B_4L
    kw = dict(max_seq=2200, flags=pkg.FLAG_NO_PASS_KERNEL, draw_device="cuda:0")
    eng, m, _ = make_pair(shape, (1, 2), **kw)
    fresh, _, _ = make_pair(shape, (1, 2), **kw)
    try:
        toks = si.make_prompts(shape.vocab, 1, 70, seed=25)[0].tolist()
        eng.sdfp_forward_logits_static(toks[:8], 0)              # resolves the symbol on this device
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        for start, n in ((0, 40), (40, 30), (0, 1)):
            eng.sdfp_forward_logits_static(toks[start:start + n], start)
        with pytest.raises(pkg.SdfpError):                        # 64 rows at a context of 2164 tokens: refused
            eng.sdfp_forward_logits_static(toks[:64], 2100)
        torch.cuda.synchronize()
        free1, _ = torch.cuda.mem_get_info()
        assert free1 == free0
        prompt = si.make_prompts(shape.vocab, 1, 90, seed=26)     # context beyond one 64-key chunk
        for k in (4, 0):
            a = eng.sdfp_generate(prompt, k, 20)
            b = fresh.sdfp_generate(prompt, k, 20)
            assert a.tokens == b.tokens and np.array_equal(a.stats, b.stats)
    finally:
        eng.close()
        fresh.close()


def test_static_scratch_on_the_dense_path():
    """A context too wide for the whole-pass kernel decodes on the tcgen05 path, whose attention
    kernel leaves a fixed 8 partials per (row, head): the static variant must size its array for
    that and reproduce the ordinary entry point bit for bit, twice in a row."""
    eng, m, _ = make_pair(si.TINY_BF16, (1, 2), max_seq=160, max_batch=4, k_max=4)
    try:
        toks = si.make_prompts(m.vocab, 1, 100, seed=27)[0].tolist()
        for start, n in ((0, 72), (72, 9)):
            ref = eng.sdfp_forward_logits(toks[start:start + n], start)
            got = eng.sdfp_forward_logits_static(toks[start:start + n], start)
            assert np.array_equal(got.view(np.uint32), ref.view(np.uint32))
    finally:
        eng.close()
