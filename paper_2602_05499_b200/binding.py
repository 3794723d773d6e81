"""ctypes binding of libsdfp.so: the same entry points as include/sdfp.h, argument
marshalling only.  Every step of the decode path runs in the library's CUDA kernels;
PyTorch is used for device memory and the stream.  There is no fallback: if the
library cannot be loaded or there is no CUDA device, calls raise."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np

from .build import LIB_PATH

SDFP_F32, SDFP_BF16 = 0, 1
FLAG_NO_GRAPH, FLAG_NO_PDL, FLAG_FMA_GEMM, FLAG_NO_PASS_KERNEL, FLAG_NO_DENSE = 1, 2, 4, 8, 16

EXPORTS = ["sdfp_create", "sdfp_set_draft_layers", "sdfp_set_draft_sublayers", "sdfp_set_draft_kv_sharing", "sdfp_generate", "sdfp_forward_logits",
           "sdfp_forward_logits_static", "sdfp_get_timing", "sdfp_time_linear", "sdfp_time_pass",
           "sdfp_debug_expire_next_wait", "sdfp_fit_scores", "sdfp_last_error", "sdfp_destroy"]


class SdfpConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("max_seq", C.c_int32), ("max_batch", C.c_int32), ("k_max", C.c_int32),
                ("dtype", C.c_int32), ("eos_id", C.c_int32), ("flags", C.c_uint32)]


class SdfpWeights(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("wq", C.POINTER(C.c_void_p)), ("wk", C.POINTER(C.c_void_p)),
                ("wv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("w_gate", C.POINTER(C.c_void_p)), ("w_up", C.POINTER(C.c_void_p)),
                ("w_down", C.POINTER(C.c_void_p)),
                ("attn_norm", C.POINTER(C.c_void_p)), ("ffn_norm", C.POINTER(C.c_void_p))]


class SdfpRoundStat(C.Structure):
    _fields_ = [("drafted", C.c_int32), ("accepted", C.c_int32), ("committed", C.c_int32)]


class SdfpTiming(C.Structure):
    _fields_ = [("prefill_ms", C.c_float), ("decode_ms", C.c_float), ("n_rounds", C.c_int32),
                ("n_draft_passes", C.c_int32), ("n_target_passes", C.c_int32),
                ("kernel_launches", C.c_int64), ("weight_bytes", C.c_int64), ("kv_bytes", C.c_int64),
                ("tokens_committed", C.c_int64)]


class SdfpError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"sdfp error {code}: {msg}")
        self.code = code


_lib = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """dlopen the library and declare the prototypes.  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise OSError(f"{p} not found: build it with paper_2602_05499_b200.build.build_library()")
    lib = C.CDLL(p)
    vp = C.c_void_p
    lib.sdfp_create.argtypes = [C.POINTER(SdfpConfig), C.POINTER(SdfpWeights), vp, C.POINTER(vp)]
    lib.sdfp_create.restype = C.c_int
    lib.sdfp_set_draft_layers.argtypes = [vp, C.POINTER(C.c_uint8)]
    lib.sdfp_set_draft_layers.restype = C.c_int
    lib.sdfp_set_draft_sublayers.argtypes = [vp, C.POINTER(C.c_uint8), C.POINTER(C.c_uint8)]
    lib.sdfp_set_draft_sublayers.restype = C.c_int
    lib.sdfp_set_draft_kv_sharing.argtypes = [vp, C.c_int32]
    lib.sdfp_set_draft_kv_sharing.restype = C.c_int
    lib.sdfp_generate.argtypes = [vp, C.POINTER(C.c_int32), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                  C.c_float, C.c_uint64, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                  C.POINTER(SdfpRoundStat), C.c_int32, C.POINTER(C.c_int32)]
    lib.sdfp_generate.restype = C.c_int
    lib.sdfp_forward_logits.argtypes = [vp, C.c_int32, C.POINTER(C.c_int32), C.c_int32, C.c_int32,
                                        C.POINTER(C.c_float)]
    lib.sdfp_forward_logits.restype = C.c_int
    lib.sdfp_forward_logits_static.argtypes = lib.sdfp_forward_logits.argtypes
    lib.sdfp_forward_logits_static.restype = C.c_int
    lib.sdfp_get_timing.argtypes = [vp, C.POINTER(SdfpTiming)]
    lib.sdfp_get_timing.restype = C.c_int
    lib.sdfp_time_linear.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_float),
                                     C.POINTER(C.c_int64)]
    lib.sdfp_time_linear.restype = C.c_int
    lib.sdfp_time_pass.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_float),
                                   C.POINTER(C.c_int64)]
    lib.sdfp_time_pass.restype = C.c_int
    lib.sdfp_debug_expire_next_wait.argtypes = [vp, C.c_uint64]
    lib.sdfp_debug_expire_next_wait.restype = C.c_int
    lib.sdfp_fit_scores.argtypes = [C.POINTER(SdfpConfig), C.POINTER(SdfpWeights), vp, C.POINTER(C.c_int32), C.c_int32, C.c_int32,
                                    C.POINTER(C.c_double), C.POINTER(C.c_double)]
    lib.sdfp_fit_scores.restype = C.c_int
    lib.sdfp_last_error.argtypes = [vp]
    lib.sdfp_last_error.restype = C.c_char_p
    lib.sdfp_destroy.argtypes = [vp]
    lib.sdfp_destroy.restype = None
    if path is None:
        _lib = lib
    return lib


def _marshal(shape, weights: Dict, max_seq: int, max_batch: int, k_max: int, eos_id: int, flags: int):
    """(SdfpConfig, SdfpWeights, objects that must stay alive) for a dict of CUDA tensors."""
    import torch
    want = torch.float32 if shape.dtype == "f32" else torch.bfloat16
    L = shape.n_layers

    def ptr(t):
        if not t.is_cuda or t.dtype != want or not t.is_contiguous():
            raise ValueError("weights must be contiguous CUDA tensors of the model's storage type")
        return t.data_ptr()

    arrs = {}
    for name in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "ffn_norm"):
        arrs[name] = (C.c_void_p * L)(*[ptr(weights["layers"][l][name]) for l in range(L)])
    w = SdfpWeights(ptr(weights["tok_embed"]), ptr(weights["final_norm"]), ptr(weights["lm_head"]),
                    *[C.cast(arrs[n], C.POINTER(C.c_void_p)) for n in
                      ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "ffn_norm")])
    cfg = SdfpConfig(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn,
                     shape.vocab, shape.rms_eps, shape.rope_theta, max_seq, max_batch, k_max,
                     SDFP_F32 if shape.dtype == "f32" else SDFP_BF16, eos_id, flags)
    return cfg, w, arrs


def sdfp_fit_scores(shape, weights: Dict, calib) -> "tuple":
    """Stage A of Algorithm 1 on the GPU: (T_l, FIT_l) per layer over the calibration sequences
    `calib` (int array [n_seq, seq_len]).  Argument marshalling only."""
    import torch
    if not torch.cuda.is_available():
        raise RuntimeError("no CUDA device: the SDFP library has no CPU path")
    lib = load_library()
    cfg, w, keep = _marshal(shape, weights, 8, 1, 0, -1, 0)
    t = np.ascontiguousarray(np.asarray(calib, dtype=np.int32))
    if t.ndim != 2:
        raise ValueError("calib must be [n_seq, seq_len]")
    trace = np.zeros(shape.n_layers, dtype=np.float64)
    fit = np.zeros(shape.n_layers, dtype=np.float64)
    torch.cuda.current_stream().synchronize()
    rc = lib.sdfp_fit_scores(C.byref(cfg), C.byref(w), C.c_void_p(torch.cuda.current_stream().cuda_stream),
                             t.ctypes.data_as(C.POINTER(C.c_int32)), t.shape[0], t.shape[1],
                             trace.ctypes.data_as(C.POINTER(C.c_double)), fit.ctypes.data_as(C.POINTER(C.c_double)))
    if rc != 0:
        raise SdfpError(rc, lib.sdfp_last_error(None).decode())
    del keep
    return trace.tolist(), fit.tolist()


class GenOutput:
    def __init__(self, tokens: List[List[int]], stats: np.ndarray, n_rounds: int, timing: Dict):
        self.tokens = tokens          # per sequence, the generated ids
        self.stats = stats            # int32 [n_rounds, batch, 3] = drafted, accepted, committed
        self.n_rounds = n_rounds
        self.timing = timing

    @property
    def acceptance_rate(self) -> float:
        d = int(self.stats[:, :, 0].sum())
        return float(self.stats[:, :, 1].sum()) / d if d else float("nan")

    @property
    def mean_committed(self) -> float:
        live = self.stats[:, :, 2] > 0
        return float(self.stats[:, :, 2].sum()) / max(1, int(live.sum()))


class Sdfp:
    """One library context.  `weights` is a dict of CUDA torch tensors laid out like
    synth_inputs.make_weights: tok_embed, lm_head, final_norm and a list `layers` of
    dicts wq, wk, wv, wo, w_gate, w_up, w_down, attn_norm, ffn_norm."""

    def __init__(self, shape, weights: Dict, max_seq: int, max_batch: int = 1, k_max: int = 8,
                 eos_id: int = -1, flags: int = 0, stream=None):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("no CUDA device: the SDFP library has no CPU path")
        self.lib = load_library()
        self.shape = shape
        self._stream = stream if stream is not None else torch.cuda.Stream()
        cfg, w, self._keep = _marshal(shape, weights, max_seq, max_batch, k_max, eos_id, flags)
        self.cfg = cfg
        handle = C.c_void_p()
        # the caller's tensors were produced on torch's current stream
        torch.cuda.current_stream().synchronize()
        rc = self.lib.sdfp_create(C.byref(cfg), C.byref(w), C.c_void_p(self._stream.cuda_stream), C.byref(handle))
        if rc != 0:
            raise SdfpError(rc, self.lib.sdfp_last_error(None).decode())
        self.handle = handle

    def _check(self, rc: int):
        if rc != 0:
            raise SdfpError(rc, self.lib.sdfp_last_error(self.handle).decode())

    def close(self):
        if getattr(self, "handle", None):
            self.lib.sdfp_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sdfp_set_draft_layers(self, keep_mask: Sequence[int]):
        m = np.ascontiguousarray(np.asarray(keep_mask, dtype=np.uint8))
        if m.shape != (self.shape.n_layers,):
            raise ValueError("keep_mask must have n_layers entries")
        self._check(self.lib.sdfp_set_draft_layers(self.handle, m.ctypes.data_as(C.POINTER(C.c_uint8))))

    def sdfp_set_draft_sublayers(self, keep_attn: Sequence[int], keep_ffn: Sequence[int]):
        a = np.ascontiguousarray(np.asarray(keep_attn, dtype=np.uint8))
        f = np.ascontiguousarray(np.asarray(keep_ffn, dtype=np.uint8))
        if a.shape != (self.shape.n_layers,) or f.shape != (self.shape.n_layers,):
            raise ValueError("both masks must have n_layers entries")
        self._check(self.lib.sdfp_set_draft_sublayers(self.handle, a.ctypes.data_as(C.POINTER(C.c_uint8)),
                                                      f.ctypes.data_as(C.POINTER(C.c_uint8))))

    def sdfp_set_draft_kv_sharing(self, share: bool):
        self._check(self.lib.sdfp_set_draft_kv_sharing(self.handle, 1 if share else 0))

    def sdfp_generate(self, prompts, k: int, max_new: int, temperature: float = 0.0, seed: int = 0) -> GenOutput:
        p = np.ascontiguousarray(np.asarray(prompts, dtype=np.int32))
        if p.ndim == 1:
            p = p[None, :]
        batch, plen = p.shape
        out = np.empty((batch, max_new), dtype=np.int32)
        out_len = np.zeros(batch, dtype=np.int32)
        max_rounds = max_new + 1
        stats = np.zeros((max_rounds, batch, 3), dtype=np.int32)
        n_rounds = C.c_int32(0)
        self._check(self.lib.sdfp_generate(
            self.handle, p.ctypes.data_as(C.POINTER(C.c_int32)), batch, plen, k, max_new,
            C.c_float(temperature), C.c_uint64(seed), out.ctypes.data_as(C.POINTER(C.c_int32)),
            out_len.ctypes.data_as(C.POINTER(C.c_int32)), stats.ctypes.data_as(C.POINTER(SdfpRoundStat)),
            max_rounds, C.byref(n_rounds)))
        toks = [out[b, :out_len[b]].tolist() for b in range(batch)]
        return GenOutput(toks, stats[:n_rounds.value].copy(), n_rounds.value, self.sdfp_get_timing())

    def sdfp_forward_logits(self, tokens: Sequence[int], start: int, draft: bool = False) -> np.ndarray:
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        out = np.empty((len(t), self.shape.vocab), dtype=np.float32)
        self._check(self.lib.sdfp_forward_logits(self.handle, 1 if draft else 0,
                                                 t.ctypes.data_as(C.POINTER(C.c_int32)), len(t), start,
                                                 out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def sdfp_forward_logits_static(self, tokens: Sequence[int], start: int, draft: bool = False) -> np.ndarray:
        """sdfp_forward_logits with the attention scratch in the library's static device array:
        for callers that must not reach a device allocator.  Same arguments, same logits."""
        t = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        out = np.empty((len(t), self.shape.vocab), dtype=np.float32)
        self._check(self.lib.sdfp_forward_logits_static(self.handle, 1 if draft else 0,
                                                        t.ctypes.data_as(C.POINTER(C.c_int32)), len(t), start,
                                                        out.ctypes.data_as(C.POINTER(C.c_float))))
        return out

    def sdfp_get_timing(self) -> Dict:
        t = SdfpTiming()
        self._check(self.lib.sdfp_get_timing(self.handle, C.byref(t)))
        return {f: getattr(t, f) for f, _ in SdfpTiming._fields_}

    def sdfp_time_linear(self, which: int, rows: int, iters: int):
        ms = C.c_float(0)
        nbytes = C.c_int64(0)
        self._check(self.lib.sdfp_time_linear(self.handle, which, rows, iters, C.byref(ms), C.byref(nbytes)))
        return ms.value, nbytes.value

    def sdfp_debug_expire_next_wait(self, wait_limit_ns: int):
        self._check(self.lib.sdfp_debug_expire_next_wait(self.handle, C.c_uint64(wait_limit_ns)))

    def sdfp_time_pass(self, draft: bool, rows: int, position: int, iters: int):
        """(ms per launch of the whole-pass kernel, bytes such a launch has to move)."""
        ms = C.c_float(0)
        nbytes = C.c_int64(0)
        self._check(self.lib.sdfp_time_pass(self.handle, 1 if draft else 0, rows, position, iters, C.byref(ms),
                                            C.byref(nbytes)))
        return ms.value, nbytes.value
