"""CPU-side checks of the C-ABI library: it builds, loads, exports every symbol the
header declares, and refuses to compute without a CUDA device (no CPU fallback)."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

import paper_2602_05499_b200 as pkg
from paper_2602_05499_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    pkg.build_library()
    return pkg.load_library()


def test_exports_match_header(lib):
    hdr = open(os.path.join(ROOT, "include", "sdfp.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(sdfp_[a-z_]+)\s*\(", hdr))
    assert declared == set(pkg.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_struct_sizes_match_header():
    assert C.sizeof(binding.SdfpConfig) == 14 * 4
    assert C.sizeof(binding.SdfpRoundStat) == 12
    assert C.sizeof(binding.SdfpWeights) == 12 * 8
    assert C.sizeof(binding.SdfpTiming) == 5 * 4 + 4 + 4 * 8      # 5 words, padding, 4 int64


def test_create_rejects_bad_arguments(lib):
    h = C.c_void_p()
    assert lib.sdfp_create(None, None, None, C.byref(h)) == -1
    assert b"NULL" in lib.sdfp_last_error(None)
    cfg = binding.SdfpConfig(4, 256, 4, 60, 688, 2048, 1e-5, 1e4, 128, 1, 4, 0, -1, 0)
    w = binding.SdfpWeights()
    assert lib.sdfp_create(C.byref(cfg), C.byref(w), None, C.byref(h)) == -1
    assert b"head_dim" in lib.sdfp_last_error(None)
    cfg.head_dim = 64
    cfg.vocab = 2050
    assert lib.sdfp_create(C.byref(cfg), C.byref(w), None, C.byref(h)) == -1
    cfg.vocab = 2048
    cfg.max_batch = 16
    cfg.k_max = 8       # 16 * 9 rows > 64
    assert lib.sdfp_create(C.byref(cfg), C.byref(w), None, C.byref(h)) == -1
    cfg.max_batch, cfg.k_max = 1, 4
    assert lib.sdfp_create(C.byref(cfg), C.byref(w), None, C.byref(h)) == -1     # NULL weight pointers
    assert b"weight" in lib.sdfp_last_error(None)


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a machine without a GPU")
def test_no_cpu_fallback(lib):
    """Without a CUDA device the library fails with SDFP_ECUDA instead of computing on the host."""
    cfg = binding.SdfpConfig(4, 256, 4, 64, 688, 2048, 1e-5, 1e4, 128, 1, 4, 0, -1, 0)
    dummy = (C.c_void_p * 4)(*[1, 1, 1, 1])
    pp = C.cast(dummy, C.POINTER(C.c_void_p))
    w = binding.SdfpWeights(1, 1, 1, pp, pp, pp, pp, pp, pp, pp, pp, pp)
    h = C.c_void_p()
    assert lib.sdfp_create(C.byref(cfg), C.byref(w), None, C.byref(h)) == -3
    assert b"no CUDA device" in lib.sdfp_last_error(None)
    import synth_inputs as si
    with pytest.raises(RuntimeError):
        pkg.Sdfp(si.TINY, {}, max_seq=64)


def test_null_context_calls_are_errors(lib):
    assert lib.sdfp_set_draft_layers(None, None) == -1
    assert lib.sdfp_get_timing(None, None) == -1
    lib.sdfp_destroy(None)
