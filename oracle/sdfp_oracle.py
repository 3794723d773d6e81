"""CPU oracle for the speculative-decode hot path of SDFP (Algorithm 1, Stage B).

TEST INFRASTRUCTURE.  Plain, slow, obviously-correct PyTorch CPU code.  Only
the tests, the smoke check and the benchmark's CPU-baseline leg may import it;
the CUDA library never does, and this file imports nothing from the library.

What it computes
  * the Llama-style decoder forward the paper's experiments presuppose
    ("LLaMA-2 family", Section IV-A): RMSNorm, rotary embeddings, multi-head
    causal attention, SwiGLU FFN, untied lm-head, no biases;
  * the draft model of Algorithm 1 ("construct draft model by removing layers
    in P"): the same weights with the layers of the prune set treated as the
    identity on the residual stream;
  * plain autoregressive decoding (the "vanilla" baseline of Table I);
  * the speculative loop of Algorithm 1 Stage B with the accept rule of Eq. 2
    and the corrected distribution of Eq. 3, greedy and sampled.

Readings taken where the paper is silent or garbled (each also listed in the
design notes of the repository):
  R1  Eq. 3 is printed as r(y) ∝ p(y) − α_j q(y); that expression can be
      negative and does not make the sampler lossless, which the paragraph
      right after it claims.  The rule of the work it cites (Leviathan et al.)
      is used: r(y) = max(0, p(y) − q(y)) / Σ max(0, p − q).  If the sum is 0
      (p ≡ q; a rejection then has probability 0) r falls back to p.
  R2  Every round emits exactly one token beyond the accepted prefix: from r at
      the first rejection j < k, from the target's distribution after the k-th
      draft when all k were accepted.  (Algorithm 1 only says "if none accepted,
      sample from f_θ"; Section II-A evaluates i = 0..k−1 only.)
  R3  Greedy decoding: a draft token is accepted iff it equals the target's
      argmax; the extra token is the target's argmax.  Ties → lowest token id.
  R4  Temperature T divides the logits of both models; no top-p / top-k.
  R5  Random numbers: see oracle/philox.py.  A categorical draw with weights w
      takes the smallest y with Σ_{y'≤y} w(y') > u·Σ w (token-id order, fp64).
  R6  Rotary pairing is (i, i + head_dim/2); angles are built in fp64 and
      rounded to the compute type; ε is added to the mean square inside the
      square root.
  R7  Storage types: for a bf16 model the weights are bf16 values (widened
      exactly) and K/V are rounded to bf16 (RNE) when they enter the cache;
      everything else is computed in `dtype` (fp32 by default, fp64 on request).
  R8  The draft keeps its own KV cache for the kept layers.  After a round in
      which all k drafts were accepted, the k-th draft token was never fed to
      the draft, so the next round's first draft call feeds two tokens.
  R9  Acceptance rate α = Σ accepted / Σ drafted over the run; a round's
      `committed` counts tokens appended after truncation to max_new / EOS.
  R10 Sub-layer pruning (Section IV-A, implementation details: attention layers and FFN
      layers are pruned at separate ratios): a decoder layer is two residual blocks,
      h += Attn(norm(h)) and h += FFN(norm(h)); the draft may drop either one on its
      own, and a dropped block is the identity on the residual stream.  `layers` lists
      the layers whose attention block runs, `ffn_layers` those whose FFN block runs
      (None = the same list: whole layers, as in Algorithm 1).
  R11 KV sharing (Section III-C: the draft is architecture-compatible with the target,
      "enabling efficient KV reuse during verification"): optionally the draft keeps no
      cache of its own.  For the committed prefix it attends the TARGET's K/V in the
      layers it runs; the K/V of the tokens it drafts go into the same cache behind the
      committed length, where the verification pass overwrites them.  Then no prompt
      pass of the draft exists and every round's first draft call feeds one token.
      With a prune set that is a suffix of the stack the two modes coincide exactly.

Pins: see tests/test_oracle_*.py.  The absolute values of the forward pass are
pinned by an independently written no-cache recomputation, hand-computable
unit cases and invariants — the paper prints no worked numerical example.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import torch

from . import philox


# ----------------------------------------------------------------------------
# building blocks
# ----------------------------------------------------------------------------

def rmsnorm(h: torch.Tensor, gain: torch.Tensor, eps: float) -> torch.Tensor:
    """x̂ = h / sqrt(mean(h²) + ε) · g   (R6)."""
    ms = (h * h).mean(dim=-1, keepdim=True)
    return h / torch.sqrt(ms + eps) * gain


def rope_angles(head_dim: int, theta: float, positions: Sequence[int], dtype) -> Tuple[torch.Tensor, torch.Tensor]:
    """cos, sin of pos · θ^(−2i/head_dim), i = 0..head_dim/2−1; fp64 then rounded (R6)."""
    half = head_dim // 2
    i = torch.arange(half, dtype=torch.float64)
    inv_freq = torch.pow(torch.tensor(theta, dtype=torch.float64), -2.0 * i / head_dim)
    pos = torch.tensor(list(positions), dtype=torch.float64)
    ang = pos[:, None] * inv_freq[None, :]
    return torch.cos(ang).to(dtype), torch.sin(ang).to(dtype)


def apply_rope(x: torch.Tensor, cos: torch.Tensor, sin: torch.Tensor) -> torch.Tensor:
    """x: [T, H, hd]; cos, sin: [T, hd/2].  Pair (i, i+hd/2) is rotated by the angle of i."""
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    c, s = cos[:, None, :], sin[:, None, :]
    return torch.cat([x1 * c - x2 * s, x2 * c + x1 * s], dim=-1)


def silu(x: torch.Tensor) -> torch.Tensor:
    return x / (1.0 + torch.exp(-x))


def _lin(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """x · Wᵀ with W [out, in] widened exactly to the compute type."""
    return x @ w.to(x.dtype).t()


def _store_round(t: torch.Tensor, kv_bf16: bool) -> torch.Tensor:
    return t.to(torch.bfloat16).to(t.dtype) if kv_bf16 else t


@dataclass
class Model:
    """Weights plus the hyper-parameters the forward needs."""
    w: Dict
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rms_eps: float
    rope_theta: float
    kv_bf16: bool
    dtype: torch.dtype = torch.float32

    @staticmethod
    def from_shape(shape, w: Dict, dtype=torch.float32) -> "Model":
        return Model(w, shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim,
                     shape.d_ffn, shape.vocab, shape.rms_eps, shape.rope_theta,
                     kv_bf16=(shape.dtype == "bf16"), dtype=dtype)


# ----------------------------------------------------------------------------
# O4: brute force — whole sequence recomputed from scratch, no cache
# ----------------------------------------------------------------------------

def forward_nocache(m: Model, tokens: Sequence[int], layers: Optional[Sequence[int]] = None,
                    ffn_layers: Optional[Sequence[int]] = None) -> torch.Tensor:
    """Logits [T, vocab] for every position of `tokens`, recomputing everything.

    `layers` = the layers that run (None = all = the target); the others are
    the identity on the residual stream (Algorithm 1: draft = layers removed).
    `ffn_layers` (R10) = the layers whose FFN block runs when that differs from
    the layers whose attention block runs.
    Written with torch ops that autograd understands (the FIT oracle
    differentiates through it).
    """
    T = len(tokens)
    H, hd = m.n_heads, m.head_dim
    attn_run = set(range(m.n_layers) if layers is None else layers)
    ffn_run = attn_run if ffn_layers is None else set(ffn_layers)
    run = sorted(attn_run | ffn_run)
    tok = torch.tensor(list(tokens), dtype=torch.long)
    h = m.w["tok_embed"].to(m.dtype)[tok]
    cos, sin = rope_angles(hd, m.rope_theta, range(T), m.dtype)
    future = torch.triu(torch.ones(T, T, dtype=torch.bool), diagonal=1)
    for l in run:
        lw = m.w["layers"][l]
        if l in attn_run:
            x = rmsnorm(h, lw["attn_norm"].to(m.dtype), m.rms_eps)
            q = apply_rope(_lin(x, lw["wq"]).view(T, H, hd), cos, sin)
            k = apply_rope(_lin(x, lw["wk"]).view(T, H, hd), cos, sin)
            v = _lin(x, lw["wv"]).view(T, H, hd)
            k, v = _store_round(k, m.kv_bf16), _store_round(v, m.kv_bf16)
            s = torch.einsum("thd,shd->hts", q, k) / math.sqrt(hd)
            s = s.masked_fill(future[None], float("-inf"))
            p = torch.softmax(s, dim=-1)
            a = torch.einsum("hts,shd->thd", p, v).reshape(T, H * hd)
            h = h + _lin(a, lw["wo"])
        if l in ffn_run:
            x = rmsnorm(h, lw["ffn_norm"].to(m.dtype), m.rms_eps)
            h = h + _lin(silu(_lin(x, lw["w_gate"])) * _lin(x, lw["w_up"]), lw["w_down"])
    return _lin(rmsnorm(h, m.w["final_norm"].to(m.dtype), m.rms_eps), m.w["lm_head"])


# ----------------------------------------------------------------------------
# O1: forward with a KV cache (one sequence)
# ----------------------------------------------------------------------------

class CachedLM:
    """One sequence, one model (target: all layers; draft: kept layers), one KV cache.

    feed(tokens, start) runs the given tokens at positions start.. and returns
    their logits [len, vocab].  Feeding at `start` overwrites the cache from
    `start` on — that is the O(1) rollback: entries beyond the committed length
    are simply never read again before being rewritten.
    """

    def __init__(self, m: Model, layers: Optional[Sequence[int]] = None, max_seq: int = 4096,
                 ffn_layers: Optional[Sequence[int]] = None):
        self.m = m
        self.layers = list(range(m.n_layers)) if layers is None else list(layers)   # attention blocks that run
        self.ffn_layers = set(self.layers if ffn_layers is None else ffn_layers)    # FFN blocks that run (R10)
        self.max_seq = max_seq
        self.k = {l: torch.zeros(max_seq, m.n_heads, m.head_dim, dtype=m.dtype) for l in self.layers}
        self.v = {l: torch.zeros(max_seq, m.n_heads, m.head_dim, dtype=m.dtype) for l in self.layers}
        self.n_feed_rows = 0  # bookkeeping for the timing leg of the benchmark

    @torch.no_grad()
    def feed(self, tokens: Sequence[int], start: int) -> torch.Tensor:
        m = self.m
        T, H, hd = len(tokens), m.n_heads, m.head_dim
        assert start + T <= self.max_seq
        self.n_feed_rows += T
        tok = torch.tensor(list(tokens), dtype=torch.long)
        h = m.w["tok_embed"][tok].to(m.dtype)
        cos, sin = rope_angles(hd, m.rope_theta, range(start, start + T), m.dtype)
        # row t (position start+t) may attend keys 0..start+t
        key_pos = torch.arange(start + T)
        row_pos = torch.arange(start, start + T)
        hidden = key_pos[None, :] > row_pos[:, None]            # [T, start+T]
        for l in sorted(set(self.layers) | self.ffn_layers):
            lw = m.w["layers"][l]
            if l in self.k:
                x = rmsnorm(h, lw["attn_norm"].to(m.dtype), m.rms_eps)
                q = apply_rope(_lin(x, lw["wq"]).view(T, H, hd), cos, sin)
                k = apply_rope(_lin(x, lw["wk"]).view(T, H, hd), cos, sin)
                v = _lin(x, lw["wv"]).view(T, H, hd)
                self.k[l][start:start + T] = _store_round(k, m.kv_bf16)
                self.v[l][start:start + T] = _store_round(v, m.kv_bf16)
                K = self.k[l][:start + T]
                V = self.v[l][:start + T]
                s = torch.einsum("thd,shd->hts", q, K) / math.sqrt(hd)
                s = s.masked_fill(hidden[None], float("-inf"))
                p = torch.softmax(s, dim=-1)
                a = torch.einsum("hts,shd->thd", p, V).reshape(T, H * hd)
                h = h + _lin(a, lw["wo"])
            if l in self.ffn_layers:
                x = rmsnorm(h, lw["ffn_norm"].to(m.dtype), m.rms_eps)
                h = h + _lin(silu(_lin(x, lw["w_gate"])) * _lin(x, lw["w_up"]), lw["w_down"])
        return _lin(rmsnorm(h, m.w["final_norm"].to(m.dtype), m.rms_eps), m.w["lm_head"])


def sharing_draft(target: "CachedLM", layers: Sequence[int], ffn_layers: Optional[Sequence[int]] = None) -> "CachedLM":
    """A draft model over `target`'s weights that reads and writes the target's cache (R11):
    the per-layer K/V tensors of the layers it runs ARE the target's tensors."""
    d = CachedLM(target.m, layers, max_seq=1, ffn_layers=ffn_layers)
    d.max_seq = target.max_seq
    d.k = {l: target.k[l] for l in d.layers}
    d.v = {l: target.v[l] for l in d.layers}
    return d


class StatelessLM:
    """Same interface as CachedLM, but every call recomputes the whole prefix
    with forward_nocache.  `history` must be supplied by the caller through
    `feed` calls that start at 0 or extend what was fed before."""

    def __init__(self, m: Model, layers: Optional[Sequence[int]] = None, memo: Optional[dict] = None):
        self.m, self.layers = m, layers
        self.toks: List[int] = []
        self.memo = memo

    @torch.no_grad()
    def feed(self, tokens: Sequence[int], start: int) -> torch.Tensor:
        assert start <= len(self.toks)
        self.toks = self.toks[:start] + [int(t) for t in tokens]
        key = tuple(self.toks)
        if self.memo is not None and key in self.memo:
            full = self.memo[key]
        else:
            full = forward_nocache(self.m, self.toks, self.layers)
            if self.memo is not None:
                self.memo[key] = full
        return full[start:start + len(tokens)]


# ----------------------------------------------------------------------------
# token decisions
# ----------------------------------------------------------------------------

def argmax_lowest(logits: torch.Tensor) -> int:
    """Index of the maximum; the lowest index among exact ties (R3)."""
    mx = logits.max()
    return int(torch.nonzero(logits == mx)[0, 0])


def softmax_T(logits: torch.Tensor, temperature: float) -> torch.Tensor:
    """softmax(logits / T) in fp64 (R4)."""
    z = logits.to(torch.float64) / temperature
    z = z - z.max()
    e = torch.exp(z)
    return e / e.sum()


def categorical(weights: torch.Tensor, u: float) -> int:
    """Smallest y with cumulative weight > u · total (R5); weights need not be normalised."""
    w = weights.to(torch.float64)
    c = torch.cumsum(w, dim=0)
    total = float(c[-1])
    hit = torch.nonzero(c > u * total)
    if hit.numel() == 0:              # only by rounding at the very top
        return int(torch.nonzero(w > 0)[-1, 0])
    return int(hit[0, 0])


def residual_distribution(p: torch.Tensor, q: torch.Tensor) -> torch.Tensor:
    """Eq. 3 under reading R1: max(0, p − q), normalised; p if that is all zero."""
    r = torch.clamp(p - q, min=0.0)
    s = r.sum()
    if float(s) <= 0.0:
        return p.clone()
    return r / s


@dataclass
class RoundStat:
    drafted: int
    accepted: int
    committed: int


@dataclass
class GenResult:
    tokens: List[int]
    rounds: List[RoundStat] = field(default_factory=list)

    @property
    def acceptance_rate(self) -> float:
        d = sum(r.drafted for r in self.rounds)
        return (sum(r.accepted for r in self.rounds) / d) if d else float("nan")

    @property
    def mean_committed(self) -> float:
        return (sum(r.committed for r in self.rounds) / len(self.rounds)) if self.rounds else float("nan")


# ----------------------------------------------------------------------------
# O2: autoregressive decoding (the "vanilla" row of Table I)
# ----------------------------------------------------------------------------

def ar_generate(target, prompt: Sequence[int], max_new: int, temperature: float = 0.0,
                seed: int = 0, seq: int = 0, eos_id: int = -1) -> GenResult:
    """Feed the prompt, then one token per step.  `target` has .feed(tokens, start)."""
    y = [int(t) for t in prompt]
    n0 = len(y)
    if n0 > 1:
        target.feed(y[:-1], 0)
    out: List[int] = []
    while len(out) < max_new:
        n = len(y)
        logits = target.feed([y[-1]], n - 1)[0]
        if temperature == 0.0:
            t = argmax_lowest(logits)
        else:
            t = categorical(softmax_T(logits, temperature),
                            philox.draw_u(seed, seq, n, philox.PURPOSE_EXTRA))
        y.append(t)
        out.append(t)
        if eos_id >= 0 and t == eos_id:
            break
    return GenResult(out)


# ----------------------------------------------------------------------------
# O3: the speculative loop (Algorithm 1, Stage B; Section II-A)
# ----------------------------------------------------------------------------

def spec_generate(target, draft, prompt: Sequence[int], k: int, max_new: int,
                  temperature: float = 0.0, seed: int = 0, seq: int = 0,
                  eos_id: int = -1, share_kv: bool = False) -> GenResult:
    """Speculative decoding with a draft that is the target minus some layers.

    State between rounds: committed tokens y[0..n−1]; the target's cache holds
    positions 0..n−2; the draft's cache holds 0..n−2 or, after a fully accepted
    round, 0..n−3 (R8).  share_kv (R11): `draft` was made by sharing_draft(target, ...);
    it has no prompt pass and feeds only the last committed token at the start of a round.
    """
    assert k >= 1
    y = [int(t) for t in prompt]
    n0 = len(y)
    if n0 > 1:
        target.feed(y[:-1], 0)
        if not share_kv:
            draft.feed(y[:-1], 0)
    draft_cached = n0 - 1            # number of committed positions in the draft cache
    res = GenResult([])
    greedy = (temperature == 0.0)
    while len(res.tokens) < max_new:
        n = len(y)
        # (i) draft k tokens autoregressively (Eq. 1)
        d: List[int] = []
        qs: List[torch.Tensor] = []
        logits = draft.feed(y[draft_cached:], draft_cached)[-1]
        for i in range(1, k + 1):
            if greedy:
                tok = argmax_lowest(logits)
            else:
                q = softmax_T(logits, temperature)
                qs.append(q)
                tok = categorical(q, philox.draw_u(seed, seq, n - 1 + i, philox.PURPOSE_DRAFT))
            d.append(tok)
            if i < k:
                logits = draft.feed([tok], n - 1 + i)[0]
        # (ii) one target pass over k+1 rows: row i gives the distribution of the token after it
        tl = target.feed([y[-1]] + d, n - 1)
        # (iii) accept token by token (Eq. 2), stop at the first rejection
        j = 0
        ps: List[torch.Tensor] = []
        while j < k:
            if greedy:
                ok = (d[j] == argmax_lowest(tl[j]))
            else:
                p = softmax_T(tl[j], temperature)
                ps.append(p)
                u = philox.draw_u(seed, seq, n + j, philox.PURPOSE_ACCEPT)
                # u < min(1, p/q)  <=>  u·q < p   (q(d) > 0 because d was drawn from q)
                ok = (u * float(qs[j][d[j]]) < float(p[d[j]]))
            if not ok:
                break
            j += 1
        # (iv) the extra token (R2)
        if greedy:
            extra = argmax_lowest(tl[j])
        else:
            u = philox.draw_u(seed, seq, n + j, philox.PURPOSE_EXTRA)
            if j < k:
                extra = categorical(residual_distribution(ps[j], qs[j]), u)
            else:
                extra = categorical(softmax_T(tl[k], temperature), u)
        # (v) commit, truncated to max_new and at EOS (R9)
        new = d[:j] + [extra]
        room = max_new - len(res.tokens)
        new = new[:room]
        if eos_id >= 0 and eos_id in new:
            new = new[:new.index(eos_id) + 1]
        y.extend(new)
        res.tokens.extend(new)
        res.rounds.append(RoundStat(k, j, len(new)))
        # (vi) roll back: the target cache is valid through n−1+j = len(y)−2 when
        # nothing was truncated; the draft was fed y[n−1], d_1..d_{k−1}.
        draft_cached = min(n + j, n + k - 1, len(y) - 1)
        if share_kv:
            draft_cached = len(y) - 1   # the target's cache holds every committed position but the last
        if eos_id >= 0 and new and new[-1] == eos_id:
            break
    return res


def keep_layers(n_layers: int, skip: Sequence[int]) -> List[int]:
    s = set(int(x) for x in skip)
    return [l for l in range(n_layers) if l not in s]
