#!/usr/bin/env python
"""Benchmark of the stairs validation pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfg2|cfg3|cfg4]

One step = one stairs_validate call (stair rows, embedding, every layer, LM head, argmax,
accept) on the validation-microbench model (24 layers, d_model 1024, vocab 32128, bf16) with a
2048-token prefix already in the KV cache and k = 8 drafted tokens (9 rows).  Prints ONE JSON
line.  With --gpus N > 1 (under torchrun) every rank runs an independent replica: requests do
not interact, so there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2407_19947_b200 import workloads as wl  # noqa: E402

METRIC = "stairs_validate_us_per_call"
UNIT = "us/call"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return {"hbm_gbs": FALLBACK_HBM_GBS}, "fallback"


def pick_workload(name: str):
    """(workload, prefix tokens in the cache, draft length k, requests per call)"""
    idx = {"cfg2": 2, "cfg3": 3, "cfg4": 4, "cfg5": 5}[name]
    w = wl.workload(idx)
    if idx == 2:
        prefix, k, n_req = 2048, 8, 1
    elif idx == 3:
        prefix, k, n_req = 512, 4, 1
    elif idx == 4:
        prefix, k, n_req = 1024, 8, 1
    else:
        prefix, k, n_req = 16384, 8, 4     # four long requests validated in one call (36 stair rows)
    return w, prefix, k, n_req


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.rows, self.proc = index, [], None

    def run(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            for line in self.proc.stdout:
                self.rows.append([c.strip() for c in line.split(",")])
        except Exception:
            pass

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
        self.join(timeout=2)
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = set()
        for r in self.rows:
            for i, n in enumerate(names):
                if len(r) > 4 + i and r[4 + i].lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_bytes(shape, prefix: int, k: int, n_req: int = 1) -> int:
    """Bytes one validate call must move: every weight matrix once plus each request's visible K/V once."""
    return shape.weight_bytes_per_call() + n_req * shape.kv_bytes_per_token() * (prefix + k + 1)


def oracle_row_seconds(w, tsrc, prompt, draft, rows):
    """Times the CPU oracle (as it stands) on the given stair rows; returns seconds per row."""
    from oracle import stairs_oracle as so
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    all_rows = so.stairs_rows(prompt, draft)
    t0 = time.perf_counter()
    toks = [so.argmax_lowest(so.forward_logits(tgt, all_rows[r])) for r in rows]
    return (time.perf_counter() - t0) / len(rows), toks


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def max_over_ranks(values, world, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (the job's time is its slowest rank's)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def kernel_source_hash() -> str:
    """Hash of the kernel sources; a stored DRAM-traffic figure is only quoted while it matches."""
    import hashlib
    h = hashlib.sha1()
    d = os.path.join(ROOT, "paper_2407_19947_b200", "csrc")
    for f in sorted(os.listdir(d)):
        with open(os.path.join(d, f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def stored_traffic(workload_name: str):
    """dram bytes per launch from the committed ncu capture of this workload, or None when the
    kernels changed since it was taken."""
    p = os.path.join(ROOT, "profiles", "traffic_k_forward.txt")
    if not os.path.exists(p):
        return None
    with open(p) as f:
        t = json.load(f)
    e = t.get(workload_name)
    if not e or e.get("kernel_source_hash") != kernel_source_hash():
        return None
    return e.get("dram_bytes_per_launch")


def time_validate(eng, torch, k, drafts_dev, steps, warmup):
    """us per stairs_validate call (commit=0) with CUDA events on the engine's stream."""
    tt = torch.zeros((1, eng.k_max + 1), dtype=torch.int32, device=eng.device)
    al = torch.zeros((1,), dtype=torch.int32, device=eng.device)
    n = drafts_dev.shape[0]
    for i in range(warmup):
        eng.validate([0], [k], drafts_dev[i % n], commit=False, out=(tt, al))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(eng.stream)
    for i in range(steps):
        eng.validate([0], [k], drafts_dev[i % n], commit=False, out=(tt, al))
    e1.record(eng.stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / steps


def workload_label(w, prefix, k, n_req):
    """One string for both arms, so the two lines name the same workload."""
    return f"{w.name}: prefix {prefix}, k {k}, {n_req * (k + 1)} stair rows, {n_req} request{'s' if n_req > 1 else ''} per call, commit=0"


def prefill_flops(shape, n_tokens: int) -> float:
    """Useful floating-point operations of one model's prefill of n_tokens positions: every layer
    matrix once per token (2 flops per weight) plus causal attention (scores and weighted values)."""
    es = 2 if shape.wdtype == wl.WDTYPE_BF16 else 4
    layer_params = (shape.weight_bytes_per_call() // es - shape.vocab * shape.d_model)     # without the LM head
    gemm = 2.0 * layer_params * n_tokens
    attn = 4.0 * shape.n_layers * shape.n_heads * shape.head_dim * (n_tokens * (n_tokens + 1) / 2.0)
    return gemm + attn


def timed_prefill(eng, torch, req, prompt):
    """ms of stairs_prefill (both models) with CUDA events on the engine's stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(eng.stream)
    eng.prefill(req, prompt)
    e1.record(eng.stream)
    eng.sync()
    return e0.elapsed_time(e1)


def forced_acceptance_sweep(eng, torch, w, prompt, cont, kf, n_gen, seed):
    """Tokens/s of the validate loop alone (no draft model) with drafts taken from the known greedy
    continuation `cont`, each drafted token corrupted with probability 1 - alpha."""
    out = {}
    rng = np.random.default_rng(seed)
    vocab = w.target.vocab
    for alpha in (0.0, 0.5, 0.8, 1.0):
        eng.prefill(0, prompt)
        produced, calls = 0, 0
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        while produced < n_gen:
            want = np.array(list(cont[produced:produced + kf]) + [0] * kf, dtype=np.int32)[:kf]
            bad = rng.random(kf) >= alpha
            want = np.where(bad, (want + 1) % vocab, want).astype(np.int32)
            _, acc = eng.validate_host([0], [kf], want[None], commit=True)
            produced += int(acc[0]) + 1
            calls += 1
        dt = time.perf_counter() - t0
        out[f"alpha_{alpha}"] = {"tokens_per_s": produced / dt, "validate_calls": calls, "tokens_per_call": produced / calls}
    return out


def generation_point(eng, prompt, k, n_new):
    out, st = eng.generate(0, prompt, k, n_new)
    decode_ms = st["total_ms"] - st["prefill_ms"]
    return out, {"tokens_per_s": n_new / (decode_ms * 1e-3), "acceptance": st["accepted"] / max(st["drafted"], 1),
                 "iterations": st["iterations"], "draft_ms": st["draft_ms"], "validate_ms": st["validate_ms"],
                 "prefill_ms": st["prefill_ms"]}


def extra_workload(idx, torch, stairs, local_rank, peak, tflops_peak):
    """Validate latency, prefill and generation of one of the larger configs, on a fresh context."""
    w, prefix, k, n_req = pick_workload(f"cfg{idx}")
    shape = w.target
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    n_new = w.max_new
    eng = stairs.Stairs(tsrc, dsrc, max_requests=n_req, max_seq_len=prefix + n_new + 16, k_max=8 if idx != 3 else 4,
                        kv_page_tokens=64, device_index=local_rank)
    res = {"workload": workload_label(w, prefix, k, n_req)}
    try:
        reqs = list(range(n_req))
        prompts = [wl.prompt_tokens(w, request=r, n=prefix + 1) for r in reqs]
        pre_ms = [timed_prefill(eng, torch, r, prompts[r]) for r in reqs]
        fl = sum(prefill_flops(shape, prefix) + prefill_flops(w.draft, prefix) for _ in reqs)
        res["prefill"] = {"ms_per_request": float(np.mean(pre_ms)), "tokens_per_s": prefix / (float(np.mean(pre_ms)) * 1e-3),
                          "useful_tflops": fl / (sum(pre_ms) * 1e-3) / 1e12,
                          "frac_of_bf16_sustained_peak": fl / (sum(pre_ms) * 1e-3) / 1e12 / tflops_peak if tflops_peak else None,
                          "note": "target and assistant, 64 positions per pass of the persistent kernel (weights re-streamed every pass; "
                                  "operands are bf16 hi+lo pairs, so the tensor pipe does twice the useful work)"}
        # validate latency per k (uniform random drafts: the time does not depend on the accept length)
        rng = np.random.default_rng(6)
        per_k = {}
        for kk in ((0, 1, 2, 4, 8) if idx == 4 else (k,)):
            dd = torch.from_numpy(rng.integers(0, shape.vocab, size=(n_req, eng.k_max)).astype(np.int32)).to(eng.device)
            tt = torch.zeros((n_req, eng.k_max + 1), dtype=torch.int32, device=eng.device)
            al = torch.zeros((n_req,), dtype=torch.int32, device=eng.device)
            n_it = 30 if idx != 5 else 15
            for _ in range(3):
                eng.validate(reqs, [kk] * n_req, dd, commit=False, out=(tt, al))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record(eng.stream)
            for _ in range(n_it):
                eng.validate(reqs, [kk] * n_req, dd, commit=False, out=(tt, al))
            e1.record(eng.stream)
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / n_it
            ab = algorithmic_bytes(shape, prefix, kk, n_req)
            per_k[f"k{kk}"] = {"us_per_call": us, "hbm_gbs": ab / (us * 1e-6) / 1e9, "frac_of_measured_peak": ab / (us * 1e-6) / 1e9 / peak,
                               "frac_of_nominal_8TBs": ab / (us * 1e-6) / 1e9 / NOMINAL_HBM_GBS}
        res["validate"] = per_k
        # every logit of one call finite (a guard against silently skipped work)
        dd = torch.from_numpy(rng.integers(0, shape.vocab, size=(n_req, eng.k_max)).astype(np.int32)).to(eng.device)
        _, _, lg = eng.validate(reqs, [k] * n_req, dd, want_logits=True)
        eng.sync()
        res["logits_finite"] = bool(torch.isfinite(lg).all())
        del lg
        if idx in (3, 4):
            gen_prompt = prompts[0][:prefix]
            out0, g0 = generation_point(eng, gen_prompt, 0, n_new)
            res["prefill"]["generate_prefill_ms"] = g0["prefill_ms"]
            gen = {"k0": g0}
            for kk in ((1, 2, 3, 4, 5, 6, 7, 8) if idx == 4 else (k,)):
                outk, gk = generation_point(eng, gen_prompt, kk, n_new)
                gk["identical_to_k0"] = outk == out0
                gk["speedup_vs_k0"] = gk["tokens_per_s"] / g0["tokens_per_s"]
                gen[f"k{kk}"] = gk
            res["generation"] = {"prompt": len(gen_prompt), "new_tokens": n_new, "per_k": gen}
            res["forced_acceptance_k4"] = forced_acceptance_sweep(eng, torch, w, gen_prompt, out0, 4, min(n_new, 96), 7)
    finally:
        eng.close()
        del eng
        tsrc.drop_cache(); dsrc.drop_cache()
        torch.cuda.empty_cache()
    return res


def run_reference(args, rank, world):
    """The oracle timed on the host cores.  Each step is one stair row (an independent no-cache
    fp32 forward) at a prefix shortened so that the whole run stays within a few minutes; the
    reported us/call scales the mean row time linearly in tokens to the full prefix and
    multiplies by the k+1 rows of a call."""
    if rank != 0:
        return
    from oracle import stairs_oracle as so
    w, prefix, k, n_req = pick_workload(args.workload)
    tsrc, _ = wl.make_sources(w, backend="numpy")
    tgt = so.OracleModel(w.target, tsrc, keep=True)
    prompt = list(wl.prompt_tokens(w, n=prefix + 1))
    draft = list(wl.uniform_tokens(k, w.target.vocab, 77))
    so.forward_logits(tgt, prompt[:16])                      # widens the weights once
    t0 = time.perf_counter()
    so.forward_logits(tgt, prompt[:64])
    t64 = time.perf_counter() - t0
    budget = args.ref_seconds / max(args.steps + args.warmup, 1)
    p_s = int(max(16, min(prefix + 1, 64 * budget / max(t64, 1e-4))))
    times = []
    for i in range(args.warmup + args.steps):
        r = i % (k + 1)
        row = prompt[:p_s] + draft[:r]
        t0 = time.perf_counter()
        so.argmax_lowest(so.forward_logits(tgt, row))
        if i >= args.warmup:
            times.append((time.perf_counter() - t0) * (prefix + 1 + r) / len(row))
    row_s = float(np.mean(times))
    value = row_s * (k + 1) * n_req * 1e6
    sample = (f"{args.steps} stair rows at prefix {p_s} of {prefix + 1}, one no-cache fp32 forward each, "
              f"scaled linearly in tokens to the full prefix and to {n_req * (k + 1)} rows per call")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": float(np.mean(times)) * 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": workload_label(w, prefix, k, n_req)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_ours(args, rank, local_rank, world):
    import torch
    from paper_2407_19947_b200 import build, stairs
    if rank == 0:
        build.build()
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
        dist.barrier()
    w, prefix, k, n_req = pick_workload(args.workload)
    if args.layers > 0:
        import dataclasses
        w = dataclasses.replace(w, name=f"{w.name}_first{args.layers}layers", target=w.target.replace(n_layers=args.layers),
                                draft_layers=min(w.draft_layers, args.layers))
    shape = w.target
    tsrc, dsrc = wl.make_sources(w, backend="torch-cuda")
    torch.cuda.set_device(local_rank)
    max_seq = prefix + 256 if shape.pos == wl.POS_ROPE else min(prefix + 256, shape.max_pos)
    eng = stairs.Stairs(tsrc, dsrc, max_requests=n_req, max_seq_len=max_seq, k_max=k, kv_page_tokens=64,
                        device_index=local_rank)
    reqs = list(range(n_req))
    prompts = [wl.prompt_tokens(w, request=r, n=prefix + 1) for r in reqs]   # prefix in the cache + the last committed token
    prompt = prompts[0]
    for r in reqs:
        eng.prefill(r, prompts[r])
    eng.sync()
    # forced drafts (first a tokens equal the target's own continuation, then a mismatch), per request
    n_var = 64 if n_req == 1 else 8
    a_list = wl.forced_accept_lengths(k, n_var * n_req, 1234)
    drafts = np.zeros((n_var, n_req, k), np.int32)
    for r in reqs:
        cont = []
        for _ in range(k + 1):                   # k+1 plain greedy steps, then roll the request back
            t_host, _ = eng.validate_host([r], [0], None, commit=True)
            cont.append(int(t_host[0, 0]))
        eng.truncate(r, len(prompts[r]))
        for i in range(n_var):
            drafts[i, r] = wl.forced_draft(np.array(cont), a_list[i * n_req + r], shape.vocab, 50 + i * n_req + r)
    d_dev = torch.from_numpy(drafts).to(eng.device)
    tt = torch.zeros((n_req, k + 1), dtype=torch.int32, device=eng.device)
    al = torch.zeros((n_req,), dtype=torch.int32, device=eng.device)
    stream = eng.stream

    def step(i):
        eng.validate(reqs, [k] * n_req, d_dev[i % n_var], commit=False, out=(tt, al))

    # accept lengths must come out as forced (checks the path end to end before timing it)
    for i in range(min(8, n_var)):
        step(i)
        eng.sync()
        got = [int(x) for x in al.cpu()]
        assert got == a_list[i * n_req:(i + 1) * n_req], (got, a_list[i * n_req:(i + 1) * n_req])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    launches0 = eng.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = eng.launch_count() - launches0
    clocks = sampler.stop()

    # per-launch events around the weight-streaming GEMMs, over the same steps
    eng.profile(True)
    gemm_ms, gemm_n, call_ms = 0.0, 0, 0.0
    for i in range(0 if args.timed_only else args.steps):
        step(i)
        g, n, c = eng.profile_read()
        gemm_ms += g
        gemm_n += n
        call_ms += c
    eng.profile(False)

    # end to end through the host-buffer entry point (drafts in, tokens and accept length out)
    pin_d = torch.from_numpy(drafts).pin_memory()
    for i in range(0 if args.timed_only else 3):
        eng.validate_host(reqs, [k] * n_req, pin_d[i].numpy())
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for i in range(0 if args.timed_only else args.steps):
        eng.validate_host(reqs, [k] * n_req, pin_d[i % n_var].numpy())
    e2e_s = time.perf_counter() - t0

    ms, e2e_ms = max_over_ranks([ms, e2e_s * 1e3], world, eng.device)
    if rank != 0:
        return
    total_calls = args.steps * world
    us_per_call = ms * 1e3 / total_calls
    peaks, peak_kind = measured_peaks()
    peak = float(peaks["hbm_gbs"])
    wbytes = shape.weight_bytes_per_call()
    abytes = algorithmic_bytes(shape, prefix, k, n_req)
    gemm_s_per_call = gemm_ms * 1e-3 / args.steps
    if gemm_n > 0:
        dominant = "k_gemm_tc: weight-streaming GEMMs (QKV, O, MLP, LM head), one launch each"
        achieved = wbytes / gemm_s_per_call / 1e9 if gemm_s_per_call > 0 else None
        roof_timing = "per-launch CUDA events in a second pass over the same steps"
        roof_bytes = wbytes
    else:
        # the whole call is ONE kernel (k_forward): its launch duration is the step time
        dominant = "k_forward: the whole validate pass in one persistent kernel"
        achieved = abytes / (ms * 1e-3 / args.steps) / 1e9
        roof_timing = "CUDA events around the timed steps (one launch per step)"
        roof_bytes = abytes
    line = {
        "metric": METRIC, "value": us_per_call, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_label(w, prefix, k, n_req),
                   "l2": "inputs larger than L2 (weights %.2f GB per call)" % (wbytes / 1e9),
                   "replicas": world},
        "clocks": clocks,
        "gpu_launches": int(launches),
        "e2e": {"value": e2e_ms * 1e3 / total_calls, "unit": UNIT,
                "h2d_bytes_per_step": int(n_req * (k * 4 + 2 * 4) + 4), "d2h_bytes_per_step": int(n_req * ((k + 1) * 4 + 4))},
        "roofline": {"bound": "hbm", "kernel": dominant, "bytes_per_launch": roof_bytes,
                     "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak if achieved else None,
                     "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS if achieved else None,
                     "peak_kind": f"of {peak_kind}", "traffic": stored_traffic(w.name) if gemm_n == 0 else None,
                     "launches_per_call": (gemm_n if gemm_n > 0 else launches) / max(args.steps, 1),
                     "timing": roof_timing},
        "call": {"algorithmic_bytes": abytes, "hbm_gbs_whole_call": abytes / (us_per_call * 1e-6) / 1e9,
                 "frac_of_measured_peak": abytes / (us_per_call * 1e-6) / 1e9 / peak,
                 "frac_of_nominal_8TBs": abytes / (us_per_call * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
                 "profiled_call_us": call_ms * 1e3 / max(args.steps, 1)},
    }
    # generation: tokens/s with stairs against k=0 greedy on the same kernels (short run)
    try:
        if args.timed_only or n_req > 1:
            raise RuntimeError('skipped (--timed-only, or a multi-request workload)')
        gen_prompt = prompt[: min(len(prompt), 512)]
        n_new = 48
        out0, st0 = eng.generate(0, gen_prompt, 0, n_new)
        outk, stk = eng.generate(0, gen_prompt, min(4, k), n_new)
        line["generation"] = {
            "prompt": len(gen_prompt), "new_tokens": n_new, "k": min(4, k),
            "greedy_tokens_per_s": n_new / ((st0["total_ms"] - st0["prefill_ms"]) * 1e-3),
            "stairs_tokens_per_s": n_new / ((stk["total_ms"] - stk["prefill_ms"]) * 1e-3),
            "acceptance": stk["accepted"] / max(stk["drafted"], 1), "identical_output": out0 == outk}
        line["generation"]["speedup_vs_k0"] = (line["generation"]["stairs_tokens_per_s"]
                                               / line["generation"]["greedy_tokens_per_s"])
    except Exception as ex:  # reported, never hidden
        line["generation"] = {"error": str(ex)}
    # the other points of the validation microbench (prefix x k), and the 7B-shaped target
    if world == 1 and not args.timed_only and not args.no_extras:
        try:
            if args.workload == "cfg2" and args.layers == 0:
                grid = {}
                rng = np.random.default_rng(5)
                for pfx in (128, 512, 2048):
                    eng.prefill(0, prompt[: pfx + 1])
                    for kk in (2, 4, 8):
                        dd = torch.from_numpy(rng.integers(0, shape.vocab, size=(16, k)).astype(np.int32)).to(eng.device)
                        us = time_validate(eng, torch, kk, dd, 100, 5)
                        ab = algorithmic_bytes(shape, pfx, kk)
                        grid[f"P{pfx}_k{kk}"] = {"us_per_call": us, "frac_of_measured_peak": ab / (us * 1e-6) / 1e9 / peak}
                line["validate_grid"] = grid
        except Exception as ex:
            line["validate_grid"] = {"error": str(ex)}
        # the larger configs, each on a fresh context: validate latency, prefill, generation
        if args.workload == "cfg2" and args.layers == 0:
            eng.close()
            eng = None
            del d_dev
            tsrc.drop_cache()
            torch.cuda.empty_cache()
            tfl = peaks.get("bf16_tflops_sustained")
            for idx in (3, 4, 5):
                try:
                    line[f"cfg{idx}"] = extra_workload(idx, torch, stairs, local_rank, peak, float(tfl) if tfl else None)
                except Exception as ex:  # reported, never hidden
                    line[f"cfg{idx}"] = {"error": f"{type(ex).__name__}: {ex}"}
    # the oracle beside it, on this host's cores, on a bounded sample
    if world == 1 and not args.no_cpu_baseline and not args.timed_only:
        cb_prefix = min(prefix, args.cpu_prefix)
        osrc = tsrc
        cb_prompt = list(prompt[: cb_prefix + 1])
        row_s, _ = oracle_row_seconds(w, osrc, cb_prompt, list(drafts[0][0]), [0])
        n_rows = int(max(1, min(k + 1, 15.0 // max(row_s, 1e-3))))
        if n_rows > 1:
            row_s, _ = oracle_row_seconds(w, osrc, cb_prompt, list(drafts[0][0]), list(range(n_rows)))
        line["cpu_baseline"] = {"value": row_s * (k + 1) * n_req * 1e6, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": f"{n_rows} of the {n_req * (k + 1)} stair rows at prefix {cb_prefix} "
                                          f"(no-cache fp32 forwards), scaled to {n_req * (k + 1)} rows"}
    print(json.dumps(line))
    if eng is not None:
        eng.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--layers", type=int, default=0,
                    help="use only the first N layers of the workload's target (small captures under a profiler)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the (prefix, k) grid and the 7B-shaped target")
    ap.add_argument("--timed-only", action="store_true",
                    help="skip the end-to-end, generation and CPU legs (short runs under a profiler)")
    ap.add_argument("--cpu-prefix", type=int, default=2048, help="prefix length of the CPU-baseline sample")
    ap.add_argument("--ref-seconds", type=float, default=120.0, help="--impl reference: time budget of the run")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    args.warmup = max(args.warmup, 3)
    run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
