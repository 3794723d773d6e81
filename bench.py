#!/usr/bin/env python
"""Benchmark of the SDFP speculative-decode path on B200.

One step = one call of sdfp_generate on the 7B-shaped workload (512-token random
prompt, 256 new tokens, greedy, draft = the model minus its 12 down-scaled layers,
k = 4): prefill of both caches, then speculative rounds until 256 tokens are
committed.  Reported:
  value     decode tokens/s over the decode phase, timed with CUDA events inside the
            library (prompt already in HBM, caches prefilled)
  e2e       tokens/s of the whole C-ABI call from host prompt to host tokens
            (host->device prompt copy, prefill, decode, device->host tokens)
  speedup   against the same library's autoregressive decode (k = 0), same run
  roofline  achieved HBM GB/s of the dominant kernel (the weight-streaming linear
            kernel) and of a whole pass, against the measured copy bandwidth
  cpu_baseline  the CPU oracle timed on a bounded sample of the same workload
With --gpus N > 1 (under torchrun) every rank runs an independent replica: the path
has no exchange step, so nothing is communicated except the timing reduction.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "decode tokens/s (batch 1, 7B-shape bf16), speedup vs AR decode, HBM % roofline"
WORKLOADS = {
    # name: (shape, n_skip, k, prompt_len, max_new, temperature, batch)
    "c2-7b-greedy-k4": (si.LLAMA7B, 12, 4, 512, 256, 0.0, 1),       # the configuration the metric is quoted on
    "c3-7b-sampled-k6": (si.LLAMA7B, 12, 6, 512, 256, 1.0, 1),      # rejection sampling, residual resampling
    "c4-13b-greedy-k4": (si.LLAMA13B, 16, 4, 2048, 512, 0.0, 1),    # long KV cache
    # the paper's own 13B setting: 50 % of the attention blocks and 35 % of the FFN blocks pruned
    "c4-13b-sublayer-k4": (si.LLAMA13B, (20, 14), 4, 2048, 512, 0.0, 1),
    "c1-tiny-greedy-k4": (si.TINY, 2, 4, 16, 64, 0.0, 1),
    "7b-4layers-greedy-k4": (si.LLAMA7B_4L, 2, 4, 64, 64, 0.0, 1),
    "7b-4layers-b8-greedy-k4": (si.LLAMA7B_4L, 2, 4, 64, 64, 0.0, 8),
    "7b-4layers-b8-long-greedy-k4": (si.LLAMA7B_4L, 2, 4, 1024, 64, 0.0, 8),   # the batch-8 context length at 4 layers
}
# batch 8 with ragged acceptance: draft length k and share of skipped layers swept
for _k in (2, 4, 8):
    for _skip in (8, 12, 16):
        WORKLOADS["c5-7b-b8-greedy-k%d-skip%d" % (_k, _skip)] = (si.LLAMA7B, _skip, _k, 1024, 256, 0.0, 8)
SEED = 20260205
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel against its
# algorithmic bytes, from an ncu capture of the kernel as it stands (None when there is none):
# measured on the 4-layer case (1076.20 MB read + 6.18 MB written against 1074.86 MB algorithmic);
# traffic grows in proportion to the layers a launch runs, so a full-size launch is taken as
# ratio x its algorithmic bytes
TRAFFIC_RATIO = 1.0070
PAPER_CONTEXT = "paper reports 1.32x-1.5x over vanilla decoding for LLaMA-2-13B/70B on unstated hardware"


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi in the background while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "200"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def skip_sets(shape, n_skip):
    """(attention blocks, FFN blocks) the draft drops; an int means whole layers."""
    if isinstance(n_skip, tuple):
        return (si.choose_skip_layers(shape.n_layers, n_skip[0]), si.choose_skip_layers(shape.n_layers, n_skip[1]))
    s = si.choose_skip_layers(shape.n_layers, n_skip)
    return s, s


def oracle_sample(shape, w_cpu, skip, k, prompt_len_sample, new_tokens, n_threads, temperature=0.0, skip_ffn=None):
    """Times the CPU oracle, as it stands, on a bounded sample: speculative greedy decode of
    `new_tokens` tokens after a `prompt_len_sample`-token prompt.  Returns tokens/s of the
    decode part (prompt pass excluded, like the GPU number) and a description."""
    import torch
    from oracle import sdfp_oracle as orc
    torch.set_num_threads(n_threads)
    m = orc.Model.from_shape(shape, w_cpu)
    prompt = si.make_prompts(shape.vocab, 1, prompt_len_sample)[0].tolist()
    cap = prompt_len_sample + new_tokens + k + 2
    tgt = orc.CachedLM(m, max_seq=cap)
    drf = orc.CachedLM(m, orc.keep_layers(shape.n_layers, skip), max_seq=cap,
                       ffn_layers=None if skip_ffn is None else orc.keep_layers(shape.n_layers, skip_ffn))
    t0 = time.perf_counter()
    tgt.feed(prompt[:-1], 0)
    drf.feed(prompt[:-1], 0)
    t1 = time.perf_counter()

    class Pre:                         # prompt pass already done: skip it inside spec_generate
        def __init__(self, lm):
            self.lm, self.first = lm, True

        def feed(self, toks, start):
            if self.first and start == 0 and len(toks) == len(prompt) - 1:
                self.first = False
                return None
            return self.lm.feed(toks, start)

    res = orc.spec_generate(Pre(tgt), Pre(drf), prompt, k, new_tokens, temperature=temperature, seed=SEED)
    t2 = time.perf_counter()
    return len(res.tokens) / (t2 - t1), t2 - t1, t1 - t0, res


def reduce_over_ranks(times, counts, device, world):
    """Replicas share nothing but this: times are reduced with MAX over ranks (the job is as slow as
    its slowest replica), counts with SUM (whole-job totals).  Works on any backend (nccl on the
    GPUs, gloo in the CPU test)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times), device=device, dtype=torch.float64)
    c = torch.tensor(list(counts), device=device, dtype=torch.float64)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], [float(x) for x in c.tolist()]


def run_reference(args, workload):
    """--impl reference: the oracle on the host cores (rank 0 only)."""
    import torch
    shape, n_skip, k, plen, n_new, temp, _batch = WORKLOADS[workload]
    skip, skip_ffn = skip_sets(shape, n_skip)
    cores = os.cpu_count() or 1
    big = shape.n_params() > 1e9
    dev = "cuda:0" if (big and torch.cuda.is_available()) else "cpu"
    w = si.make_weights(shape, skip, device=dev, skip_ffn=skip_ffn)
    w_cpu = si.weights_to(w, "cpu")
    del w
    sample_prompt, sample_new = (32, 8) if big else (plen, n_new)
    vals, secs = [], []
    for i in range(args.warmup + args.steps):
        v, dt, _, _ = oracle_sample(shape, w_cpu, skip, k, sample_prompt, sample_new, cores, temp, skip_ffn)
        if i >= args.warmup:
            vals.append(v)
            secs.append(dt)
    value = float(np.mean(vals))
    sample = f"speculative greedy decode of {sample_new} tokens after a {sample_prompt}-token prompt, k={k}"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(secs)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": {"workload": workload, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2-7b-greedy-k4", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--share-kv", action="store_true", help="the draft attends the target's KV cache (no draft cache, no draft prompt pass)")
    ap.add_argument("--flags", type=int, default=0, help="sdfp_config.flags (1 no graph, 2 no PDL, 4 FMA GEMM, 8 one kernel per operation instead of the whole-pass kernel)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, args.workload)
        return

    import torch
    import torch.distributed as dist

    import paper_2602_05499_b200 as pkg

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    pkg.build_library()

    shape, n_skip, k, plen, n_new, temp, batch = WORKLOADS[args.workload]
    skip, skip_ffn = skip_sets(shape, n_skip)
    dev = f"cuda:{local_rank}"
    w = si.make_weights(shape, skip, device=dev, skip_ffn=skip_ffn)
    eng = pkg.Sdfp(shape, w, max_seq=plen + n_new + 16, max_batch=batch, k_max=8, flags=args.flags)
    eng.sdfp_set_draft_sublayers(si.keep_mask(shape.n_layers, skip), si.keep_mask(shape.n_layers, skip_ffn))
    if args.share_kv:
        eng.sdfp_set_draft_kv_sharing(True)
    want_cpu = (rank == 0 and world == 1 and not args.no_cpu_baseline)
    w_cpu = si.weights_to(w, "cpu") if want_cpu else None
    del w
    torch.cuda.empty_cache()
    prompts = si.make_prompts(shape.vocab, batch, plen, seed=si.PROMPT_SEED + 1000 * rank)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up (also captures the round graphs) -------------------------------------------
    for _ in range(args.warmup):
        eng.sdfp_generate(prompts, k, n_new, temp, SEED)
        eng.sdfp_generate(prompts, 0, n_new, temp, SEED)

    # ---- timed: K speculative steps ---------------------------------------------------------------
    sampler = ClockSampler(local_rank)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    dec_ms = pre_ms = 0.0
    launches = tokens = 0
    wbytes = kvbytes = 0
    draft_passes = target_passes = 0
    acc, tau = [], []
    out = None
    for _ in range(args.steps):
        out = eng.sdfp_generate(prompts, k, n_new, temp, SEED)
        t = out.timing
        dec_ms += t["decode_ms"]
        pre_ms += t["prefill_ms"]
        launches += t["kernel_launches"]
        tokens += t["tokens_committed"]
        wbytes += t["weight_bytes"]
        kvbytes += t["kv_bytes"]
        draft_passes += t["n_draft_passes"]
        target_passes += t["n_target_passes"]
        acc.append(out.acceptance_rate)
        tau.append(out.mean_committed)
    e1.record()
    barrier()
    wall_s = time.perf_counter() - t0
    clocks = sampler.stop()
    step_ms = e0.elapsed_time(e1) / args.steps

    # ---- autoregressive decode with the same library (the speedup's denominator) ------------
    ar_dec_ms = 0.0
    ar_steps = max(1, min(args.steps, 3))
    ar = None
    for _ in range(ar_steps):
        ar = eng.sdfp_generate(prompts, 0, n_new, temp, SEED)
        ar_dec_ms += ar.timing["decode_ms"]
    ar_tok_s = ar_steps * batch * n_new / (ar_dec_ms * 1e-3)
    ar_t = ar.timing
    ar_pass_gbs = (ar_t["weight_bytes"] + ar_t["kv_bytes"]) / (ar_t["decode_ms"] * 1e-3) / 1e9
    if temp == 0.0:
        assert ar.tokens == out.tokens, "speculative greedy output differs from autoregressive output"

    # ---- dominant kernel, live: the whole-pass kernel (one launch = one forward pass), timed with a
    # CUDA-event pair around every launch on the library's stream; the draft pass is the launch the
    # decode phase spends most of its time in (k draft passes per verify pass)
    peak, peak_src = measured_peak_gbs()
    per_kernel = {}
    mid = plen + n_new // 2                      # a context in the middle of the generation
    uses_pass = (shape.dtype == "bf16" and not (args.flags & (pkg.FLAG_NO_PASS_KERNEL | pkg.FLAG_FMA_GEMM))
                 and batch * 9 <= 16)          # k_max = 8: wider contexts run one kernel per operation
    if uses_pass:
        for name, draft, rows in (("draft_pass@M=1", True, 1), ("draft_pass@M=2", True, 2),
                                  ("verify_pass@M=%d" % (k + 1), False, k + 1), ("ar_pass@M=1", False, 1)):
            ms, nbytes = eng.sdfp_time_pass(draft, rows, mid, 24)
            per_kernel[name] = {"us": round(ms * 1e3, 1), "GB/s": round(nbytes / ms / 1e6, 1),
                                "bytes": int(nbytes), "frac_of_peak": round(nbytes / ms / 1e6 / peak, 3)}
        dom_ms, dom_bytes = eng.sdfp_time_pass(True, 1, mid, 48)
        dom_name = "pass_kernel (draft pass: %d attention and %d FFN blocks of %d layers + lm-head, M=1, context %d)" % (
            shape.n_layers - len(skip), shape.n_layers - len(skip_ffn), shape.n_layers, mid)
    else:
        names = ["qkv", "o_proj", "gate_up", "down", "lm_head"]
        for rows in (batch, batch * (k + 1)):
            for which, nm in enumerate(names):
                ms, nbytes = eng.sdfp_time_linear(which, rows, 64 if which < 4 else 16)
                per_kernel[f"{nm}@M={rows}"] = {"us": round(ms * 1e3, 2), "GB/s": round(nbytes / ms / 1e6, 1)}
        dom_ms, dom_bytes = eng.sdfp_time_linear(2, batch * (k + 1), 128)
        dom_name = "linear kernel (gate/up, M=%d)" % (batch * (k + 1))
    kernel_gbs = dom_bytes / dom_ms / 1e6

    # ---- reduce over ranks --------------------------------------------------------------------------
    (dec_ms_max, step_ms_max, wall_max), (tokens_all, launches_all) = reduce_over_ranks(
        [dec_ms, step_ms, wall_s], [float(tokens), float(launches)], dev, world)
    value = tokens_all / (dec_ms_max * 1e-3)
    e2e_value = tokens_all / wall_max
    spec_pass_gbs = (wbytes + kvbytes) / (dec_ms * 1e-3) / 1e9

    cpu_baseline = None
    if want_cpu:
        cores = os.cpu_count() or 1
        big = shape.n_params() > 1e9
        sp, sn = (32, 8) if big else (plen, n_new)
        v, dt, pre_dt, _ = oracle_sample(shape, w_cpu, skip, k, sp, sn, cores, temp, skip_ffn)
        cpu_baseline = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                        "sample": f"speculative greedy decode of {sn} tokens after a {sp}-token prompt, k={k}, "
                                  f"{dt:.1f} s (+ {pre_dt:.1f} s prompt pass)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms_max, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if shape.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape.name, "batch": batch, "prompt_len": plen,
                       "max_new": n_new, "k": k, "skip_layers": skip, "skip_ffn_blocks": skip_ffn,
                       "decoding": "greedy" if temp == 0.0 else "sampled, temperature %g, Philox seed %d" % (temp, SEED),
                       "l2": "inputs larger than L2 (weights %.1f GB per pass)" % (shape.n_params() * 2 / 1e9)
                       if shape.dtype == "bf16" else "tiny model: launch-bound, weights fit in L2",
                       "replicas": world, "flags": args.flags, "draft_shares_target_kv": bool(args.share_kv)},
            "speedup_vs_own_ar": value / world / ar_tok_s,
            "ar_tokens_per_s": ar_tok_s,
            "acceptance_rate": float(np.mean(acc)), "tokens_per_round": float(np.mean(tau)),
            "prefill_ms_per_step": pre_ms / args.steps,
            "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": int(prompts.nbytes),
                    "d2h_bytes_per_step": int(batch * (4 * n_new + 4 + 12 * (n_new + 1))),
                    "note": "whole sdfp_generate call: prompt copy, prefill of both caches, decode, token copy"},
            "gpu_launches": int(launches_all),
            "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": dom_name,
                         "achieved": kernel_gbs, "peak": peak, "unit": "GB/s", "frac": kernel_gbs / peak,
                         "peak_source": peak_src, "traffic": int(TRAFFIC_RATIO * dom_bytes) if uses_pass else None,
                         "algorithmic_bytes_per_launch": int(dom_bytes), "us_per_launch": dom_ms * 1e3,
                         "pass_level": {"spec_GB/s": spec_pass_gbs, "spec_frac_of_peak": spec_pass_gbs / peak,
                                        "spec_frac_of_8TB/s": spec_pass_gbs / 8000.0,
                                        "ar_GB/s": ar_pass_gbs, "ar_frac_of_peak": ar_pass_gbs / peak,
                                        "ar_frac_of_8TB/s": ar_pass_gbs / 8000.0,
                                        "draft_passes": draft_passes, "target_passes": target_passes},
                         "per_kernel": per_kernel},
            "cpu_baseline": cpu_baseline,
            "context": PAPER_CONTEXT,
        }
        print(json.dumps(line))
    eng.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
