#!/usr/bin/env python
"""Benchmark of the review-step hot path: generated tokens/s of the cascade on the decoder-only
workload (7B-shaped target, 68M-shaped draft, Max-Gram below; 128-token prompt, 256 new tokens,
greedy, k = 4), plus the review-step HBM figures.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one whole generation (prefill + all cascade steps) of one sequence per GPU.  With
N > 1 (torchrun) every rank runs an independent replica on its own prompt: no data-path
collective, weak scaling; the barrier and the max-over-ranks time use torch.distributed.
`--impl reference` times the CPU oracle (a deliberately plain program) on a bounded sample of
the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

PROMPT_LEN, MAX_NEW, MAX_BLOCK = 128, 256, 4
K_MATRIX = [[4, 0], [0, 4]]
WORKLOAD = "llama7b-shaped target + 68M-shaped draft + Max-Gram, prompt 128, generate 256, greedy, K=[[4,0],[0,4]]"
METRIC = "generated tokens/s and review-step HBM GB/s (% of 8 TB/s) at 1 B200"
TRAFFIC_RATIO = 1.040                  # DRAM bytes / weight bytes of the tensor-core GEMM, from its ncu capture
ORACLE_PROMPT, ORACLE_NEW = 8, 4       # bounded CPU sample: same models, 8-token prompt, 4 new tokens


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        self.thread.join(timeout=2)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def build_inputs(rank: int, device: str):
    import workloads
    ts, ds = workloads.SHAPES["llama7b"], workloads.SHAPES["draft68m"]
    tb = workloads.make_weights(ts, seed=100, device=device)
    db = workloads.make_weights(ds, seed=101, device=device)
    prompt = workloads.make_prompt(ts.vocab, PROMPT_LEN, seed=1000 + rank)
    nxt = workloads.bigram_table(prompt, ts.vocab, seed=7)
    return ts, ds, tb, db, prompt, nxt


def oracle_sample(ts, ds, tb, db, prompt, nxt):
    """One bounded oracle run: returns (tokens, seconds)."""
    import oracle
    oracle.build()
    t0 = time.time()
    oms = [oracle.Model(ts, oracle.blob_to_u16(tb)), oracle.Model(ds, oracle.blob_to_u16(db))]
    load_s = time.time() - t0
    p = prompt[:ORACLE_PROMPT]
    t0 = time.time()
    toks, _, _ = oracle.cascade_generate(oms, p, nxt, K_MATRIX, MAX_BLOCK, p, ORACLE_NEW)
    dt = time.time() - t0
    for m in oms:
        m.close()
    return len(toks), dt, load_s


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    device = "cuda" if torch.cuda.is_available() else "cpu"
    ts, ds, tb, db, prompt, nxt = build_inputs(0, device)
    import oracle
    oracle.build()
    oms = [oracle.Model(ts, oracle.blob_to_u16(tb)), oracle.Model(ds, oracle.blob_to_u16(db))]
    del tb, db
    p = prompt[:ORACLE_PROMPT]
    times, tokens = [], 0
    for i in range(args.warmup + args.steps):
        t0 = time.time()
        toks, _, _ = oracle.cascade_generate(oms, p, nxt, K_MATRIX, MAX_BLOCK, p, ORACLE_NEW)
        if i >= args.warmup:
            times.append(time.time() - t0)
            tokens += len(toks)
    total = sum(times)
    value = tokens / total
    cores = len(os.sched_getaffinity(0))
    sample = f"{ORACLE_PROMPT}-token prompt, {ORACLE_NEW} new tokens per step, same models and cascade"
    # the oracle's own time for the two calls of a review step: one 5-row target forward over the
    # sample's cache, and one accept call on its logits (one row, k = 4, greedy)
    blk = prompt[ORACLE_PROMPT:ORACLE_PROMPT + MAX_BLOCK + 1]
    t0 = time.time()
    logits = oms[0].review_forward(blk, ORACLE_PROMPT)
    review_s = time.time() - t0
    t0 = time.time()
    oracle.spec_accept(logits[None, :, :], None, np.asarray(blk[:MAX_BLOCK])[None, :], 0.0)
    accept_s = time.time() - t0
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(len(times), 1),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sample": sample},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0, "oracle_review_forward_s": review_s, "oracle_accept_s": accept_s}
    print(json.dumps(line), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the product path has no CPU fallback")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    from paper_2312_11462_b200 import binding as b
    from paper_2312_11462_b200.dist import aggregate_tokens_per_s

    ts, ds, tb, db, prompt, nxt = build_inputs(rank, "cuda")
    target, draft = b.Model(ts, tb), b.Model(ds, db)
    nxt_dev = torch.from_numpy(nxt).cuda()
    casc = b.Cascade([target, draft], K_MATRIX, MAX_BLOCK, nxt_dev, PROMPT_LEN)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        casc.csd_cascade_generate(prompt, prompt, MAX_NEW)
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    stats = []
    for _ in range(args.steps):
        toks, st = casc.csd_cascade_generate(prompt, prompt, MAX_NEW)
        assert len(toks) == MAX_NEW
        stats.append(st)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    barrier()
    bracket_ms = ev0.elapsed_time(ev1)
    device_ms = sum(s["prefill_ms"] + s["decode_ms"] for s in stats)
    tokens = MAX_NEW * args.steps
    value, e2e, ms_per_step = aggregate_tokens_per_s(tokens, device_ms, bracket_ms, args.steps,
                                                     dist if world > 1 else None)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    st = stats[-1]
    reviews = st["reviews"]
    h2d = 2 * 4 * PROMPT_LEN
    d2h = 4 * MAX_NEW + 8 * sum(reviews)
    # ---- review-step figures on the target: m = k+1 = 5 rows over a committed 128-token cache
    blk = torch.from_numpy(prompt[:MAX_BLOCK + 1]).cuda()
    logits = torch.empty(MAX_BLOCK + 1, ts.vocab, device="cuda")
    n_rev = 30
    for _ in range(3):
        target.csd_review_forward(blk, PROMPT_LEN, logits)
    torch.cuda.synchronize()
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r0.record()
    for i in range(n_rev):
        target.csd_review_forward(blk, PROMPT_LEN + i, logits)
    r1.record()
    torch.cuda.synchronize()
    review_us = 1e3 * r0.elapsed_time(r1) / n_rev
    # kernel-class split of the same call, from event pairs around every launch
    target.csd_model_profile(True)
    for i in range(n_rev):
        target.csd_review_forward(blk, PROMPT_LEN + i, logits)
    prof = target.csd_model_profile_read()
    target.csd_model_profile(False)
    # accept kernel on the review's own logits (rows = 1, greedy)
    tok = torch.from_numpy(prompt[:MAX_BLOCK]).cuda().reshape(1, MAX_BLOCK)
    ws = b.csd_spec_accept_workspace(1, MAX_BLOCK, ts.vocab, "cuda")
    outs = (torch.empty(1, dtype=torch.int32, device="cuda"), torch.empty(1, dtype=torch.int32, device="cuda"))
    t3 = logits.reshape(1, MAX_BLOCK + 1, ts.vocab)
    for _ in range(3):
        b.csd_spec_accept(t3, None, tok, 0.0, workspace=ws, out=outs)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for _ in range(50):
        b.csd_spec_accept(t3, None, tok, 0.0, workspace=ws, out=outs)
    a1.record()
    torch.cuda.synchronize()
    accept_us = 1e3 * a0.elapsed_time(a1) / 50

    peak, peak_kind = measured_peaks()
    weight_bytes = 2.0 * (sum(int(np.prod(s)) for n, _, s in __import__("workloads").blob_layout(ts)[0]
                              if "norm" not in n and n != "embed"))
    kv_positions = PROMPT_LEN + n_rev / 2
    kv_bytes = 2.0 * 2 * ts.n_layers * ts.d_inner * kv_positions
    review_gbs = (weight_bytes + kv_bytes) / (review_us * 1e-6) / 1e9
    gemm_launch_us = 1e3 * prof["gemm_ms"] / max(prof["gemm_launches"], 1)
    gemm_gbs = prof["gemm_weight_bytes"] / (prof["gemm_ms"] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": "skinny_gemm_tc_kernel (TMA-staged weight-streaming GEMM on tcgen05, m=5)", "achieved": gemm_gbs,
                "peak": peak, "peak_kind": f"{peak_kind} STREAM-style copy", "unit": "GB/s", "frac": gemm_gbs / peak,
                "traffic": TRAFFIC_RATIO * prof["gemm_weight_bytes"] / max(prof["gemm_launches"], 1),
                "traffic_note": "dram read+write per launch = algorithmic bytes x 1.040, the ratio ncu measured over "
                                "the q|k|v / o / gate+up / down launches of one layer (profiles/skinny_gemm_tc_kernel_*)",
                "bytes_per_launch": prof["gemm_weight_bytes"] / max(prof["gemm_launches"], 1),
                "us_per_launch": gemm_launch_us}
    # the same kernel inside the pipelined forward (no event between launches, so the next launch's prologue
    # overlaps the tail of this one): the timed review forward apportioned by the bracketed shares
    class_ms = prof["gemm_ms"] + prof["attn_ms"] + prof["other_ms"]
    piped_us = review_us * prof["gemm_ms"] / class_ms
    piped_gbs = weight_bytes / piped_us / 1e3
    roofline["in_pipeline"] = {"us_per_forward": piped_us, "achieved": piped_gbs, "frac": piped_gbs / peak,
                               "note": "review forward timed as a whole x the GEMM's share of the bracketed launches"}

    # every kernel class of the review step against its own HBM roofline (event pairs around each launch,
    # so consecutive kernels do not overlap here as they do in the timed forward)
    attn_us = 1e3 * prof["attn_ms"] / n_rev
    accept_bytes = 4.0 * ts.vocab * (MAX_BLOCK + 1)
    kernel_rooflines = {
        "weight_streaming_gemm": {"bytes": weight_bytes, "us": 1e3 * prof["gemm_ms"] / n_rev, "GBps": gemm_gbs,
                                  "frac_of_8TBps": gemm_gbs / 8000.0, "frac_of_measured": gemm_gbs / peak},
        "block_attention": {"bytes": kv_bytes, "us": attn_us, "GBps": kv_bytes / attn_us / 1e3,
                            "frac_of_8TBps": kv_bytes / attn_us / 1e3 / 8000.0, "note": "latency-bound at a 128-token cache"},
        "accept": {"bytes": accept_bytes, "us": accept_us, "GBps": accept_bytes / accept_us / 1e3,
                   "frac_of_8TBps": accept_bytes / accept_us / 1e3 / 8000.0,
                   "note": "one row, greedy: latency-bound; the 64-row sweep is in `--configs accept`"},
    }

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        n_tok, dt, _ = oracle_sample(ts, ds, tb, db, prompt, nxt)
        cpu = {"value": n_tok / dt, "unit": "tokens/s", "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
               "sample": f"{ORACLE_PROMPT}-token prompt, {ORACLE_NEW} new tokens, same models and cascade ({dt:.1f} s)"}

    # a short sample of every other configuration, so that each has a figure in this line
    other = None
    if world == 1 and not args.no_configs:
        variants = cfg_variants(b, ts, tb, target, prompt, draft, nxt_dev)
        draft.close()
        other = {"variants": variants, "tiny_cascade": cfg_tiny(b),
                 "accept": [cfg_accept(b, peak, 128256, 16, 0.5), cfg_accept(b, peak, 128256, 4, 0.5),
                            cfg_accept(b, peak, 32000, 4, 0.5)],
                 "long_cache_review_step": cfg_long(b, peak, tb, reviews=6)}
        target.close()
        del casc, tb, db
        torch.cuda.empty_cache()
        other["t5xxl_target"] = cfg_t5(b, cascade=False)

    line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": "inputs (13.2 GB of weights per forward) exceed the 126 MB L2",
                       "arithmetic": "bf16 weights and K/V, fp32 activations and accumulation",
                       "replicas": world},
            "e2e": {"value": e2e, "unit": "tokens/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h},
            "gpu_launches": int(sum(s["kernel_launches"] for s in stats)),
            "clocks": clocks, "roofline": roofline, "cpu_baseline": cpu,
            "target_forwards_per_token": st["forwards"][0] / MAX_NEW,
            "decode_tokens_per_s": MAX_NEW / (st["decode_ms"] * 1e-3),
            "prefill_ms": st["prefill_ms"], "decode_ms": st["decode_ms"],
            "review_step_us": review_us, "review_hbm_gbs": review_gbs, "review_frac_of_8tbs": review_gbs / 8000.0,
            "review_frac_of_measured": review_gbs / peak,
            "review_split_us": {"gemm": 1e3 * prof["gemm_ms"] / n_rev, "attention": 1e3 * prof["attn_ms"] / n_rev,
                                "other": 1e3 * prof["other_ms"] / n_rev},
            "accept_us": accept_us, "kernel_rooflines": kernel_rooflines, "configs": other, "cascade_stats": {k: st[k] for k in ("reviews", "forwards", "drafted", "accepted",
                                                                        "mag_calls")}}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_review_only(args):
    """Profiling aid: `--review-only N` runs N review forwards (m = k+1 = 5 rows over a committed
    128-token cache) of the 7B-shaped target, optionally cut to `--layers L` layers so that a
    counter capture holds a few GB at most, then one accept call, and prints their mean times."""
    import torch
    import workloads
    from dataclasses import replace
    from paper_2312_11462_b200 import binding as b
    if args.accept_only:
        V, k = (int(x) for x in args.accept_only.split(","))
        peak, _ = measured_peaks()
        print(json.dumps(cfg_accept(b, peak, V, k, 0.5)), flush=True)
        return
    S = args.cache or PROMPT_LEN
    ts = workloads.SHAPES["llama7b" if S + 32 <= workloads.SHAPES["llama7b"].max_seq else "llama7b_long"]
    if args.layers:
        ts = replace(ts, n_layers=args.layers)
    tb = workloads.make_weights(ts, seed=100, device="cuda")
    prompt = torch.from_numpy(workloads.make_prompt(ts.vocab, S + MAX_BLOCK + 1, seed=1000)).cuda()
    target = b.Model(ts, tb)
    target.csd_prefill(prompt[:S].contiguous(), 0)              # wide passes of 128 rows
    blk = prompt[S:S + MAX_BLOCK + 1].contiguous()
    logits = torch.empty(MAX_BLOCK + 1, ts.vocab, device="cuda")
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(args.review_only):
        target.csd_review_forward(blk, S, logits)
    ev1.record()
    torch.cuda.synchronize()
    tok = blk[:MAX_BLOCK].reshape(1, MAX_BLOCK).contiguous()
    n_acc, out = b.csd_spec_accept(logits.reshape(1, MAX_BLOCK + 1, ts.vocab), None, tok, 0.0)
    torch.cuda.synchronize()
    print(json.dumps({"review_only": args.review_only, "layers": ts.n_layers,
                      "review_us": 1e3 * ev0.elapsed_time(ev1) / args.review_only,
                      "n_acc": int(n_acc[0]), "out": int(out[0])}), flush=True)


def timed_us(fn, n):
    """Mean microseconds per call of fn(i), CUDA events on the current stream."""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return 1e3 * e0.elapsed_time(e1) / n


def cfg_tiny(b):
    """Configuration 1: the tiny cascade (prompt 32, 64 new tokens, greedy, k = 4)."""
    import torch
    import workloads
    ts, ds = workloads.SHAPES["tiny_target"], workloads.SHAPES["tiny_draft"]
    tb, db = workloads.make_weights(ts, 0, "cuda"), workloads.make_weights(ds, 1, "cuda")
    prompt = workloads.make_prompt(ts.vocab, 32, seed=0)
    nxt = torch.from_numpy(workloads.bigram_table(prompt, ts.vocab, seed=0)).cuda()
    casc = b.Cascade([b.Model(ts, tb), b.Model(ds, db)], K_MATRIX, MAX_BLOCK, nxt, 32)
    for _ in range(3):
        casc.csd_cascade_generate(prompt, prompt, 64)
    t0 = time.time()
    for _ in range(10):
        toks, st = casc.csd_cascade_generate(prompt, prompt, 64)
    dt = (time.time() - t0) / 10
    return {"config": "1 tiny cascade (prompt 32, 64 new, greedy, k=4)", "tokens_per_s": 64 / dt,
            "target_forwards_per_token": st["forwards"][0] / 64, "ms_per_generation": 1e3 * dt}


def cfg_accept(b, peak, V, k, sigma, rows=64):
    """Configuration 2: one point of the stand-alone accept sweep (fp32 logits, temperature 1)."""
    import torch
    import workloads
    # two input sets, alternated, so that a call never finds its own logits in L2 when they fit
    sets = [workloads.accept_case(rows, k, V, sigma, seed=7 + j, device="cuda") for j in range(2)]
    ws = b.csd_spec_accept_workspace(rows, k, V, "cuda")
    outs = (torch.empty(rows, dtype=torch.int32, device="cuda"), torch.empty(rows, dtype=torch.int32, device="cuda"))

    def call(i):
        t, d, tok = sets[i & 1]
        b.csd_spec_accept(t, d, tok, 1.0, seed=11, step=i, workspace=ws, out=outs)
    for i in range(4):
        call(i)
    us = timed_us(call, 20)
    nbytes = 4.0 * V * (2 * k + 1) * rows
    return {"config": "2 accept sweep", "V": V, "k": k, "sigma": sigma, "rows": rows, "us": us,
            "algorithmic_MB": nbytes / 1e6, "GBps": nbytes / us / 1e3, "frac_of_8TBps": nbytes / us / 1e3 / 8000.0,
            "frac_of_measured": nbytes / us / 1e3 / peak, "mean_accepted": float(outs[0].float().mean())}


def cfg_long(b, peak, tb, block_rows=(2, 5, 9, 17), reviews=8, S=2048):
    """Configuration 5: review step (forward + accept) of the 7B-shaped target over a 2048-token cache.
    The drafted block comes from a stand-in draft whose logits are the target's own along the draft's
    path plus N(0, 0.5): the harness advances the target one token at a time (untimed) to get those
    logits, samples the drafts from them, rolls the cache length back and times the review forward and
    the accept call on the block (temperature 1).  `reviews` consecutive review steps per block size,
    each continuing from what the previous one accepted."""
    import torch
    import workloads
    ts = workloads.SHAPES["llama7b_long"]
    target = b.Model(ts, tb)
    prompt = torch.from_numpy(workloads.make_prompt(ts.vocab, S, seed=5)).cuda()
    pe = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    target.csd_prefill(prompt[:S - 1].contiguous(), 0)      # (once untimed: first use of the wide-block kernels)
    torch.cuda.synchronize()
    pe[0].record()
    target.csd_prefill(prompt[:S - 1].contiguous(), 0)
    pe[1].record()
    torch.cuda.synchronize()
    prefill_ms = pe[0].elapsed_time(pe[1])
    wbytes = 2.0 * (sum(int(np.prod(sh)) for n, _, sh in workloads.blob_layout(ts)[0] if "norm" not in n and n != "embed"))
    gen = torch.Generator(device="cuda")
    gen.manual_seed(55)
    out = []
    for m in block_rows:
        k = m - 1
        ws = b.csd_spec_accept_workspace(1, k, ts.vocab, "cuda")
        res = (torch.empty(1, dtype=torch.int32, device="cuda"), torch.empty(1, dtype=torch.int32, device="cuda"))
        logits = torch.empty(m, ts.vocab, device="cuda")
        one = torch.empty(1, ts.vocab, device="cuda")
        pos, last = S - 1, prompt[S - 1:S].clone()          # `last` is the newest token, not yet in the cache
        us_f, us_a, acc = [], [], []
        for it in range(reviews + 1):
            # the stand-in draft's path (untimed): k single-row target forwards
            toks, dl, cur = [], [], last
            for i in range(k):
                target.csd_review_forward(cur.contiguous(), pos + i, one)
                d = one + 0.5 * torch.randn(one.shape, generator=gen, device="cuda")
                cur = torch.multinomial(torch.softmax(d.double(), -1), 1, generator=gen).reshape(1).to(torch.int32)
                toks.append(cur); dl.append(d)
            block = torch.cat([last] + toks).contiguous()
            dlog = torch.cat(dl).reshape(1, k, ts.vocab).contiguous()
            dtok = torch.cat(toks).reshape(1, k).contiguous()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            torch.cuda.synchronize()
            e[0].record()
            target.csd_review_forward(block, pos, logits)                 # rolled back: the block is reviewed at once
            e[1].record()
            b.csd_spec_accept(logits.reshape(1, m, ts.vocab), dlog, dtok, 1.0, seed=9, step=it, workspace=ws, out=res)
            e[2].record()
            torch.cuda.synchronize()
            n_acc, tok = int(res[0][0]), int(res[1][0])
            if it > 0:                                                    # the first step warms up
                us_f.append(1e3 * e[0].elapsed_time(e[1])); us_a.append(1e3 * e[1].elapsed_time(e[2])); acc.append(n_acc)
            pos += n_acc + 1
            last = torch.tensor([tok], dtype=torch.int32, device="cuda")
        fwd, accept = statistics.median(us_f), statistics.median(us_a)
        kv = 2.0 * 2 * ts.n_layers * ts.d_inner * (S + m)
        nbytes = wbytes + kv + 4.0 * ts.vocab * (2 * k + 1)
        out.append({"config": "5 long-cache review step", "S": S, "m": m, "review_forward_us": fwd, "accept_us": accept,
                    "step_us": fwd + accept, "mean_accepted": sum(acc) / len(acc), "reviews": len(acc),
                    "GBps": nbytes / (fwd + accept) / 1e3, "frac_of_8TBps": nbytes / (fwd + accept) / 1e3 / 8000.0,
                    "frac_of_measured": nbytes / (fwd + accept) / 1e3 / peak, "prompt_prefill_ms": prefill_ms})
    target.close()
    return out


def cfg_variants(b, ts, tb, target, prompt, draft=None, nxt_dev=None):
    """Review-step variants on the 7B-shaped target: a tree-shaped block (the paper's tree-attention
    setting: eight candidates at the first position, the lead continued by a chain of three) and a
    batched review (three sequences of five rows in one pass over the weights)."""
    import torch
    parent = [-1] + [0] * 8 + [1, 9, 10]
    toks = torch.from_numpy(prompt[:len(parent)].copy()).cuda()
    for _ in range(3):
        lg = target.csd_review_forward_tree(toks, parent, PROMPT_LEN)
    out = torch.zeros(2 + 3 * len(parent), dtype=torch.int32, device="cuda")
    par = np.asarray(parent, dtype=np.int32)

    def tree_step(i):
        lg = target.csd_review_forward_tree(toks, parent, PROMPT_LEN)
        b._check("csd_tree_accept_greedy", b.lib.csd_tree_accept_greedy(lg.data_ptr(), toks.data_ptr(), par.ctypes.data, len(parent),
                                                                      ts.vocab, out.data_ptr(), b._stream()))
    tree_us = timed_us(tree_step, 10)
    others = [b.Model(ts, tb) for _ in range(2)]
    models = [target] + others
    blocks = [torch.from_numpy(prompt[i:i + MAX_BLOCK + 1].copy()).cuda() for i in range(3)]
    for m_ in others:
        m_.csd_prefill(torch.from_numpy(prompt[:PROMPT_LEN].copy()).cuda(), 0)
    for _ in range(3):
        b.csd_review_forward_batch(models, blocks, [PROMPT_LEN] * 3)
    batch_us = timed_us(lambda i: b.csd_review_forward_batch(models, blocks, [PROMPT_LEN] * 3), 10)
    for m_ in others:
        m_.close()
    res = {"tree_review_step": {"rows": len(parent), "shape": "8 candidates at the first position, lead + chain of 3", "us": tree_us},
           "batched_review": {"sequences": 3, "rows_each": MAX_BLOCK + 1, "us": batch_us, "us_per_sequence": batch_us / 3}}
    if draft is not None:
        # the same models under the paper's budget matrix for this pair (Appendix B: [[2,10],[0,10]]): the draft
        # reviews ten Max-Gram tokens at a time, the target two draft tokens; blocks of up to 16 drafts
        casc = b.Cascade([target, draft], [[2, 10], [0, 10]], 16, nxt_dev, PROMPT_LEN)
        casc.csd_cascade_generate(prompt, prompt, 32)
        toks, st = casc.csd_cascade_generate(prompt, prompt, MAX_NEW)
        res["paper_budget_matrix"] = {"K": [[2, 10], [0, 10]], "max_block": 16, "new_tokens": len(toks),
                                      "tokens_per_s": len(toks) / (1e-3 * (st["prefill_ms"] + st["decode_ms"])),
                                      "target_forwards_per_token": st["forwards"][0] / max(len(toks), 1),
                                      "reviews": st["reviews"], "accepted": st["accepted"], "mag_tokens": st["mag_tokens"]}
    return res


def cfg_t5(b, cascade=True):
    """Configuration 4: T5-xxl-shaped target with base- and small-shaped drafts, temperature 1."""
    import torch
    import workloads
    shapes = [workloads.SHAPES[n] for n in (("t5xxl", "t5base", "t5small") if cascade else ("t5xxl",))]
    blobs = [workloads.make_weights(sh, seed=200 + i, device="cuda") for i, sh in enumerate(shapes)]
    models = [b.Model(sh, w) for sh, w in zip(shapes, blobs)]
    enc = workloads.make_prompt(shapes[0].vocab, 256, seed=9)
    res = {"config": "4 T5-xxl-shaped target (encoder 256 tokens)"}
    if cascade:
        nxt = torch.from_numpy(workloads.bigram_table(enc, shapes[0].vocab, seed=3)).cuda()
        K = [[2, 2, 0], [0, 1, 4], [0, 0, 4]]
        casc = b.Cascade(models, K, 4, nxt, 256)
        start = np.array([0], dtype=np.int32)
        casc.csd_cascade_generate(enc, start, 128, temperature=1.0, seed=1)
        t0 = time.time()
        toks, st = casc.csd_cascade_generate(enc, start, 128, temperature=1.0, seed=2)
        dt = time.time() - t0
        res.update({"cascade": "horizontal [[2,2,0],[0,1,4],[0,0,4]], 128 new, T=1", "tokens_per_s": len(toks) / dt,
                    "prefill_ms": st["prefill_ms"], "decode_ms": st["decode_ms"],
                    "target_forwards_per_token": st["forwards"][0] / max(len(toks), 1), "reviews": st["reviews"],
                    "accepted": st["accepted"]})
    else:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        models[0].csd_encoder_forward(torch.from_numpy(enc).cuda())
        e1.record()
        torch.cuda.synchronize()
        res["encoder_ms"] = e0.elapsed_time(e1)
    blk = torch.zeros(5, dtype=torch.int32, device="cuda")
    logits = torch.empty(5, shapes[0].vocab, device="cuda")
    for _ in range(2):
        models[0].csd_review_forward(blk, 64, logits)
    res["target_review_us_m5"] = timed_us(lambda i: models[0].csd_review_forward(blk, 64, logits), 10)
    for m_ in models:
        m_.close()
    return res


def run_configs(args):
    """`--configs a,b,..` measures the other workload configurations in full (tiny cascade, accept sweep,
    T5-shaped horizontal cascade, long-cache review steps) and prints one JSON line each; the default
    bench line is configuration 3 and carries a short sample of each of them."""
    import workloads
    from paper_2312_11462_b200 import binding as b
    peak, _ = measured_peaks()
    which = set(args.configs.split(","))
    if "tiny" in which:
        print(json.dumps(cfg_tiny(b)), flush=True)
    if "accept" in which:
        for V in (4096, 32000, 128256):
            for k in (1, 2, 4, 8, 16):
                for sigma in ((0.1, 0.5, 2.0) if (V, k) == (32000, 4) else (0.5,)):
                    print(json.dumps(cfg_accept(b, peak, V, k, sigma)), flush=True)
    if "long" in which:
        tb = workloads.make_weights(workloads.SHAPES["llama7b_long"], seed=100, device="cuda")
        for line in cfg_long(b, peak, tb, reviews=32):
            print(json.dumps(line), flush=True)
        del tb
    if "t5" in which:
        print(json.dumps(cfg_t5(b, cascade=True)), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true", help="leave the samples of the other configurations out of the line")
    ap.add_argument("--review-only", type=int, default=0, help="profiling aid: only N review forwards of the target")
    ap.add_argument("--layers", type=int, default=0, help="with --review-only: cut the target to L layers")
    ap.add_argument("--cache", type=int, default=0, help="with --review-only: committed cache length (default 128)")
    ap.add_argument("--accept-only", default="", help="profiling aid: V,k of one 64-row accept case (sigma 0.5), timed alone")
    ap.add_argument("--configs", default="", help="measure other configurations: tiny,accept,long,t5")
    args = ap.parse_args()
    if args.configs:
        run_configs(args)
    elif args.review_only or args.accept_only:
        run_review_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
