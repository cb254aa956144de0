#!/usr/bin/env python
"""Benchmark of the GQLA decode hot path on B200.

A step = one pass of the absorb path (absorb_q -> decode_absorb_final -> up_proj with one piece per
sequence; absorb_q -> decode_absorb -> combine_up_proj, the split merge fused with the up-projection,
when sequences are split)
over the canonical workload (h_q=128, g=8, d_h=128, r_kv=512, d_r=64, B=64, T=4096, s_q=1,
bf16 cache).  The GQA path (decode_gqa -> combine_splits on the expanded cache, s_q=2) is
measured in the same run and reported under "paths".  One JSON line on stdout.

    python bench.py --gpus 1 --steps 50 --warmup 5
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N   (independent replicas)
    python bench.py --impl reference      (the fp64 CPU oracle on the host cores)
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2605_15250_b200 import accounting as acct
from paper_2605_15250_b200 import replicas
from paper_2605_15250_b200 import synth
from paper_2605_15250_b200.timing import ClockSampler, kernel_ms_back_to_back, kernel_sustained

METRIC = "decode attn tokens/s (absorb path, canonical config, 1 B200)"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one decode_absorb_final launch on C1 (one piece per sequence)
# (the committed ncu summary of this kernel on C1), valid for the kernel source with this digest only.
NCU_TRAFFIC = {"bytes": 311.5e6 + 4.8e6, "kernel_sha256_16": "5eb945007aae1803", "num_splits": 1}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def ncu_traffic(num_splits: int):
    """DRAM traffic of the dominant kernel from the committed ncu capture, or None when the capture was
    taken with another split plan or the kernel source has changed since."""
    import hashlib

    src = os.path.join(ROOT, "paper_2605_15250_b200", "csrc", "tc_decode_absorb.cuh")
    try:
        with open(src, "rb") as fh:
            digest = hashlib.sha256(fh.read()).hexdigest()[:16]
    except OSError:
        return None
    if digest != NCU_TRAFFIC["kernel_sha256_16"] or num_splits != NCU_TRAFFIC["num_splits"]:
        return None
    return NCU_TRAFFIC["bytes"]


def pick_splits(batch: int, units_per_seq: int, min_len: int, slots: int) -> int:
    """Smallest split count that keeps at least 80 % of the resident work slots (CTAs, or CTA pairs
    on the absorb path) busy, with >= 512 rows per split.  Every extra split costs partial traffic."""
    s = 1
    while batch * units_per_seq * s < 0.8 * slots and (min_len // (2 * s)) >= 512:
        s *= 2
    return s


# ---------------------------------------------------------------------------------- reference arm (oracle)


def oracle_tokens_per_s(w: synth.Workload, x: dict, n_seqs: int, steps: int, warmup: int):
    """Times the fp64 oracle's absorb path on the first n_seqs sequences of the workload."""
    from threadpoolctl import threadpool_info

    from oracle import gqla_oracle as O

    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    idx = list(range(n_seqs))
    ss, sl = x["seq_start"].numpy()[idx], x["seqlens"].numpy()[idx]
    n_rows = int(ss[-1] + sl[-1])

    def step():
        f_qc, f_qr = synth.to_f64(x["q_c"][idx]), synth.to_f64(x["q_r"][idx])
        return O.absorb_path(od, f_qc, f_qr, synth.to_f64(x["w_uk"]), synth.to_f64(x["w_uv"]),
                             x["cache"][:n_rows].to(torch.float64).numpy(), ss, sl, w.s_q, w.scale)

    for _ in range(warmup):
        step()
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        step()
        times.append(time.perf_counter() - t0)
    cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    per_step = sum(times) / len(times)
    return n_seqs * w.s_q / per_step, per_step, cores


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = synth.WORKLOADS["C1"]
    x = synth.make_inputs(w)
    n_seqs = w.batch  # one pass of the oracle over the whole batch takes about half a second on 16 cores
    val, per_step, cores = oracle_tokens_per_s(w, x, n_seqs, args.steps, min(args.warmup, 1))
    sample = f"all {n_seqs} sequences per step, all {w.h_q} heads, T={w.seqlen} (the whole workload)"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "C1 canonical absorb path: h_q=128 g=8 d_h=128 r_kv=512 d_r=64 B=64 T=4096 s_q=1",
                   "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------- our arm


def sustained_figures(launch, seconds: float, gpu_index: int, nbytes: float, flops: float, peaks: dict) -> dict:
    """The kernel back to back for `seconds` under whatever clock the power cap leaves: time per launch, the
    median SM clock sampled meanwhile, cycles (time x clock), and the roofline fraction against the measured
    copy bandwidth and the SUSTAINED measured matmul rate."""
    r = kernel_sustained(launch, seconds, gpu_index)
    t = r["kernel_us"] * 1e-6
    tf_sus = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    r.update({"gbs": nbytes / t / 1e9, "tflops": flops / t / 1e12,
              "frac_of_measured_sustained_roofline": acct.roofline_time(flops, nbytes, tf_sus * 1e12,
                                                                        peaks["hbm_gbs"] * 1e9) / t,
              "frac_of_nominal_roofline": acct.roofline_time(flops, nbytes, 2.25e15, 8e12) / t})
    return r


def extra_paths(dev, local_rank: int, steps: int, warmup: int, seconds: float) -> dict:
    """The other workloads of the metric (\"per path\"): the ragged LLaMA-3-8B-shaped batch (both paths, s_q = 1 and 2)
    and the long-context batch at its best split plan, each as decode-kernel time (back to back), whole-path
    time (one graph replay per step) and roofline fractions.  Their caches are drawn on the device."""
    from paper_2605_15250_b200 import sweep
    from paper_2605_15250_b200.decoder import GqlaDecoder

    import time as _time

    out = {}
    cases = {"C3": [("absorb", 1, -3), ("absorb", 2, -3), ("gqa", 1, -2), ("gqa", 2, -2)],
             "C4": [("absorb", 1, -32), ("absorb", 2, -32), ("gqa", 1, -32), ("gqa", 2, -32)]}
    for name, lst in cases.items():
        base = synth.WORKLOADS[name]
        x = synth.make_inputs(base, cache_device=dev)  # weights, lengths and the cache are shared by the cases
        dec = GqlaDecoder(base.h_q, base.g, base.d_h, base.r_kv, base.d_r, x["w_uk"].to(dev), x["w_uv"].to(dev),
                          x["cache"], x["seq_start"].to(dev), x["seqlens"].to(dev), base.scale)
        dec.expand_cache()
        for path, s_q, S in lst:
            w = base.with_(s_q=s_q)
            xq = {**x, **synth.make_queries(w)}
            _time.sleep(0.3)  # let the clocks recover from the previous case's load
            res = sweep.time_case(dec, w, xq, path, S, steps, warmup)
            if res:
                out[f"{name}_{path}_sq{s_q}"] = res
        del dec, x
        torch.cuda.empty_cache()
    return out


def fp8_paths(dec, x, x2, q2, peaks, peak_kind: str, steps: int) -> dict:
    """Both decode paths over an FP8 (E4M3) cache holding the same rows: C1 (absorb, s_q = 1) and C2 (GQA, s_q = 2).
    Per-plane scales max|x| / 448; the queries are quantised per row inside the timed chain.  The tensor roof is
    twice the measured bf16 matmul rate (no FP8 rate is measured on this machine; the nominal ratio is 2)."""
    from paper_2605_15250_b200 import binding as B

    w1, w2 = synth.WORKLOADS["C1"], synth.WORKLOADS["C2"]
    dev = dec.device
    N = dec.cache.shape[0]
    total_tokens = int(x["seqlens"].sum())
    amax = lambda t: max(float(t.float().abs().max()) / 448.0, 1e-8)
    sc, sr = amax(dec.cache[:, :w1.r_kv]), amax(dec.cache[:, w1.r_kv:])
    sk, sv = amax(dec.k_c), amax(dec.v)
    u8 = lambda *shape: torch.empty(shape, dtype=torch.uint8, device=dev)
    cache8, kc8, v8, kr8 = u8(N, w1.d_abs), u8(N, w1.g, w1.d_h), u8(N, w1.g, w1.d_h), u8(N, w1.d_r)
    B.gqla_quantize_cols_e4m3(dec.cache, w1.r_kv, sc, sr, cache8)
    B.gqla_quantize_cols_e4m3(dec.k_c, w1.d_h, sk, sk, kc8)
    B.gqla_quantize_cols_e4m3(dec.v, w1.d_h, sv, sv, v8)
    B.gqla_quantize_cols_e4m3(dec.cache[:, w1.r_kv:], w1.d_r, sr, sr, kr8)
    out = {}
    tf8 = 2.0 * peaks["bf16_tflops"]

    def entry(name, w, chain, kernel, nbytes, flops, extra):
        replay, _ = dec.capture(chain)
        for _ in range(3):
            replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            replay()
        e1.record()
        torch.cuda.synchronize()
        chain_us = e0.elapsed_time(e1) * 1e3 / steps
        k_us = kernel_ms_back_to_back(kernel, steps) * 1e3
        t = k_us * 1e-6
        t_mem, t_mma = nbytes / (peaks["hbm_gbs"] * 1e9), flops / (tf8 * 1e12)
        out[name] = {"workload": w.name, "s_q": w.s_q, "cache": "E4M3, one byte per element", "kernel_us": k_us,
                     "path_us": chain_us, "tokens_per_s": w.batch * w.s_q / (chain_us * 1e-6), "gbs": nbytes / t / 1e9,
                     "tflops": flops / t / 1e12, "algorithmic_bytes": nbytes, "flops": flops,
                     "roofline": {"bound": "hbm" if t_mem >= t_mma else "tensor", "frac": max(t_mem, t_mma) / t,
                                  "peak_hbm_gbs": peaks["hbm_gbs"], "peak_fp8_tflops": tf8,
                                  "peak_source": f"hbm of {peak_kind}; fp8 tensor = 2 x bf16 of {peak_kind} (nominal ratio)",
                                  "frac_of_nominal_roofline": acct.roofline_time(flops, nbytes, 4.5e15, 8e12) / t}, **extra}

    # absorb path: absorb_q (bf16) -> per-row quantisation -> FP8 attention (one piece per sequence) -> merge + up-projection
    q_c, q_r = x["q_c"].to(dev), x["q_r"].to(dev)
    q_hat = dec._get("q_hat", (w1.batch, w1.s_q, w1.h_q, w1.d_abs), torch.bfloat16)
    qh8, qhs = u8(*q_hat.shape), torch.empty(q_hat.shape[:-1], dtype=torch.float32, device=dev)
    o_part = dec._get("o_part_a8", (w1.batch, 1, w1.s_q, w1.h_q, w1.r_kv), torch.float32)
    lse_part = dec._get("lse_part_a8", (w1.batch, 1, w1.s_q, w1.h_q), torch.float32)
    o_out = dec._get("o_a", (w1.batch, w1.s_q, w1.h_q, w1.d_h), torch.bfloat16)

    o_hat = dec._get("o_hat", (w1.batch, w1.s_q, w1.h_q, w1.r_kv), torch.bfloat16)

    def absorb_kernel():
        B.gqla_decode_absorb_fp8_final(dec.dims, qh8, qhs, cache8, sc, dec.seq_start, dec.seqlens, dec.scale, o_hat, None,
                                       dec.status)

    def absorb_chain():
        B.gqla_absorb_q(dec.dims, q_c, q_r, dec.w_uk, q_hat)
        B.gqla_quantize_rows_e4m3(q_hat, w1.r_kv, sc, sr, qh8, qhs)
        absorb_kernel()
        B.gqla_up_proj(dec.dims, o_hat, dec.w_uv, o_out)
        return o_out

    rows1 = w1.batch * w1.s_q * w1.h_q
    nb = w1.d_abs * total_tokens + rows1 * (w1.d_abs + 4) + 2 * rows1 * w1.r_kv
    entry("absorb_fp8", w1, absorb_chain, absorb_kernel, nb, acct.absorb_flops(w1.h_q, w1.r_kv, w1.d_r, w1.s_q, total_tokens),
          {"chain": "absorb_q, quantize_rows_e4m3, decode_absorb_fp8_final, up_proj"})

    # GQA path: per-row quantisation of [q^C ; q^R] -> FP8 attention (balanced plan) -> merge
    q8, qs = u8(*q2.shape), torch.empty(q2.shape[:-1], dtype=torch.float32, device=dev)
    S_g = -2 if B.gqla_balanced_workers(dec.dims, torch.bfloat16, w2.s_q, "gqa") > 0 else 1
    og_part = dec._get("o_part_g8", (w2.batch, abs(S_g), w2.s_q, w2.h_q, w2.d_h), torch.float32)
    lg_part = dec._get("lse_part_g8", (w2.batch, abs(S_g), w2.s_q, w2.h_q), torch.float32)
    og = dec._get("o_g", (w2.batch, w2.s_q, w2.h_q, w2.d_h), torch.bfloat16)

    def gqa_kernel():
        B.gqla_decode_gqa_fp8(dec.dims, q8, qs, kc8, v8, kr8, sv, dec.seq_start, dec.seqlens, dec.scale, S_g, og_part, lg_part,
                              dec.status)

    def gqa_chain():
        B.gqla_quantize_rows_e4m3(q2, w2.d_h, sk, sr, q8, qs)
        gqa_kernel()
        B.gqla_combine_splits(og_part, lg_part, og, None)
        return og

    rows2 = w2.batch * w2.s_q * w2.h_q
    pieces = 1.25 if S_g < 0 else 1.0
    nb2 = (2 * w2.g * w2.d_h + w2.d_r) * total_tokens + rows2 * (w2.d_gqa + 4) + int(4 * rows2 * pieces * (w2.d_h + 1))
    entry("gqa_fp8", w2, gqa_chain, gqa_kernel, nb2, acct.gqa_flops(w2.h_q, w2.d_h, w2.d_r, w2.s_q, total_tokens),
          {"chain": "quantize_rows_e4m3, decode_gqa_fp8, combine_splits", "num_splits": S_g})
    dec.check_status()
    return out


def time_region(fn, steps: int, dist_on: bool):
    """Times `steps` calls of fn with CUDA events on the current stream; returns total ms (max over ranks)."""
    import torch.distributed as dist

    if dist_on:
        dist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    if dist_on:
        dist.barrier()
    return replicas.max_over_ranks(e0.elapsed_time(e1), "cuda")


def run_ours(args):
    import torch.distributed as dist

    from paper_2605_15250_b200 import binding as B
    from paper_2605_15250_b200 import build as gbuild
    from paper_2605_15250_b200.decoder import GqlaDecoder

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist_on = world > 1
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if dist_on:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        gbuild.build()
    if dist_on:
        dist.barrier()
    B.lib()
    peaks, peak_kind = load_peaks()
    steps, warmup = args.steps, max(args.warmup, 3)

    # ---- workload: replicas only -- every rank owns an independent batch (no data-path collective)
    w1 = synth.WORKLOADS["C1"].with_(seed=replicas.replica_seed(synth.WORKLOADS["C1"].seed, rank))
    x = synth.make_inputs(w1)
    dev = torch.device("cuda", local_rank)
    dec = GqlaDecoder(w1.h_q, w1.g, w1.d_h, w1.r_kv, w1.d_r, x["w_uk"].to(dev), x["w_uv"].to(dev),
                      x["cache"].to(dev), x["seq_start"].to(dev), x["seqlens"].to(dev), w1.scale)
    q_c, q_r = x["q_c"].to(dev), x["q_r"].to(dev)
    total_tokens = int(x["seqlens"].sum())
    kern_a = B.kernel_for(dec.dims, torch.bfloat16, w1.s_q, "absorb")
    n_sm = torch.cuda.get_device_properties(local_rank).multi_processor_count
    W_a = B.gqla_balanced_workers(dec.dims, torch.bfloat16, w1.s_q, "absorb")
    # Absorb path: the balanced plan pays one more 128 KB output tile per cut, so it is only taken when the
    # fixed plan with one split per sequence would leave more than a fifth of the CTA pairs idle.
    units_a = w1.batch * ((w1.s_q * w1.h_q + 127) // 128)
    if args.splits != 0:
        S_a = args.splits
    elif W_a > 0 and args.plan != "fixed" and units_a < 0.8 * (n_sm // 2):
        S_a = -3
    else:
        S_a = pick_splits(w1.batch, (w1.s_q * w1.h_q + 127) // 128, w1.seqlen, n_sm // 2)
    if S_a < 0:
        plan_a, _ = B.gqla_balanced_plan([int(t) for t in x["seqlens"]], -S_a, W_a)
        pieces_a = sum(1 for pl in plan_a for lo, hi in pl if hi > lo) / w1.batch
    else:
        pieces_a = S_a

    def absorb_step():
        dec.absorb_step(q_c, q_r, S_a)

    for _ in range(warmup):
        absorb_step()
    dec.check_status()

    # dominant kernel alone, timed live with events around each launch inside the timed region
    q_hat = dec._get("q_hat", (w1.batch, w1.s_q, w1.h_q, w1.d_abs), torch.bfloat16)
    o_part = dec._get("o_part_a", (w1.batch, abs(S_a), w1.s_q, w1.h_q, w1.r_kv), torch.float32)
    lse_part = dec._get("lse_part_a", (w1.batch, abs(S_a), w1.s_q, w1.h_q), torch.float32)
    o_hat = dec._get("o_hat", (w1.batch, w1.s_q, w1.h_q, w1.r_kv), torch.bfloat16)
    o_out = dec._get("o_a", (w1.batch, w1.s_q, w1.h_q, w1.d_h), torch.bfloat16)
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    it = {"i": 0}

    def absorb_step_instrumented():
        a, b = kev[it["i"]]
        it["i"] += 1
        B.gqla_absorb_q(dec.dims, q_c, q_r, dec.w_uk, q_hat)
        a.record()
        if S_a == 1:  # the chain GqlaDecoder.absorb_step runs with one piece per sequence
            B.gqla_decode_absorb_final(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, o_hat, None,
                                       dec.status)
            b.record()
            B.gqla_up_proj(dec.dims, o_hat, dec.w_uv, o_out)
        else:
            B.gqla_decode_absorb(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, S_a, o_part, lse_part,
                                 dec.status)
            b.record()
            B.gqla_combine_up_proj(dec.dims, o_part, lse_part, dec.w_uv, o_out, None)

    # The step as a user serves it: the four launches captured once in a CUDA graph, one replay per step
    # (the eager chain costs more host time per step than the GPU needs to run it).
    replay_absorb, _ = dec.capture(dec.absorb_step, q_c, q_r, S_a)
    for _ in range(warmup):
        replay_absorb()
    sampler = ClockSampler(local_rank)
    sampler.start()
    total_ms = time_region(replay_absorb, steps, dist_on)
    # same region, eager and with events around the dominant kernel of every step
    eager_ms = time_region(absorb_step_instrumented, steps, dist_on) / steps
    clocks = sampler.stop()
    dec.check_status()
    ms_per_step = total_ms / steps
    kern_ms = statistics.mean(a.elapsed_time(b) for a, b in kev)
    if S_a == 1:
        kern_b2b_ms = kernel_ms_back_to_back(
            lambda: B.gqla_decode_absorb_final(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, o_hat, None,
                                               dec.status), steps)
    else:
        kern_b2b_ms = kernel_ms_back_to_back(
            lambda: B.gqla_decode_absorb(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, S_a, o_part,
                                         lse_part, dec.status), steps)
    value = replicas.aggregate_tokens_per_s(world, w1.batch, w1.s_q, ms_per_step)

    kbytes = acct.decode_kernel_bytes("absorb", h_q=w1.h_q, g=w1.g, d_h=w1.d_h, r_kv=w1.r_kv, d_r=w1.d_r,
                                      s_q=w1.s_q, batch=w1.batch, total_tokens=total_tokens, num_splits=pieces_a,
                                      final=S_a == 1)
    kflops = acct.absorb_flops(w1.h_q, w1.r_kv, w1.d_r, w1.s_q, total_tokens)
    t_mem = kbytes / (peaks["hbm_gbs"] * 1e9)
    t_mma = kflops / (peaks["bf16_tflops"] * 1e12)
    gbs = kbytes / (kern_ms * 1e-3) / 1e9
    tfs = kflops / (kern_ms * 1e-3) / 1e12
    if t_mem >= t_mma:
        roof = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": gbs / peaks["hbm_gbs"]}
    else:
        roof = {"bound": "tensor", "achieved": tfs, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": tfs / peaks["bf16_tflops"]}
    roof.update({"traffic": ncu_traffic(S_a), "kernel": f"gqla_decode_absorb[{kern_a}]", "kernel_us": kern_ms * 1e3,
                 "kernel_us_back_to_back": kern_b2b_ms * 1e3, "peak_source": f"of {peak_kind}", "algorithmic_bytes": kbytes, "flops": kflops,
                 "achieved_gbs": gbs, "achieved_tflops": tfs,
                 "frac_of_roofline_time": max(t_mem, t_mma) / (kern_ms * 1e-3),
                 "frac_of_nominal_roofline": acct.roofline_time(kflops, kbytes, 2.25e15, 8e12) / (kern_ms * 1e-3)})
    # ---- end to end through the public API with host buffers: per step, the queries and the step's new
    # cache rows go host -> device from pinned memory, and the attention output comes back.
    # One pinned staging buffer [q_c | q_r | new cache rows] -> one copy each way; the copies, the scatter
    # of the new rows into the cache and the three kernels are captured together, so a step is one graph
    # launch plus the wait for its result.
    T = w1.seqlen
    cache3 = dec.cache.view(w1.batch, T, w1.d_abs)
    new_rows = x["cache"].view(w1.batch, T, w1.d_abs)[:, T - w1.s_q:, :].contiguous()
    n_qc, n_qr, n_new = x["q_c"].numel(), x["q_r"].numel(), new_rows.numel()
    h_in = torch.empty(n_qc + n_qr + n_new, dtype=torch.bfloat16).pin_memory()
    h_in[:n_qc] = x["q_c"].reshape(-1)
    h_in[n_qc:n_qc + n_qr] = x["q_r"].reshape(-1)
    h_in[n_qc + n_qr:] = new_rows.reshape(-1)
    d_in = torch.empty(n_qc + n_qr + n_new, dtype=torch.bfloat16, device=dev)
    d_qc = d_in[:n_qc].view_as(x["q_c"])
    d_qr = d_in[n_qc:n_qc + n_qr].view_as(x["q_r"])
    d_new = d_in[n_qc + n_qr:].view_as(new_rows)
    h_out = torch.empty((w1.batch, w1.s_q, w1.h_q, w1.d_h), dtype=torch.bfloat16).pin_memory()

    def e2e_body():
        d_in.copy_(h_in, non_blocking=True)
        cache3[:, T - w1.s_q:, :].copy_(d_new)
        o = dec.absorb_step(d_qc, d_qr, S_a)
        h_out.copy_(o, non_blocking=True)
        return o

    replay_e2e, _ = dec.capture(e2e_body)

    def e2e_step():
        replay_e2e()
        torch.cuda.current_stream().synchronize()  # the host reads the step's result before the next step

    for _ in range(3):
        e2e_step()
    e2e_ms = time_region(e2e_step, steps, dist_on) / steps
    e2e = {"value": replicas.aggregate_tokens_per_s(world, w1.batch, w1.s_q, e2e_ms), "unit": UNIT,
           "h2d_bytes_per_step": h_in.numel() * 2, "d2h_bytes_per_step": h_out.numel() * 2, "ms_per_step": e2e_ms}

    # the long loops come after the end-to-end region: a second at the power cap leaves the clocks low for a while
    if world == 1 and not args.no_sustained:
        if S_a == 1:
            launch_a = lambda: B.gqla_decode_absorb_final(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale,
                                                          o_hat, None, dec.status)
        else:
            launch_a = lambda: B.gqla_decode_absorb(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, S_a,
                                                    o_part, lse_part, dec.status)
        roof["sustained"] = sustained_figures(launch_a, args.sustained_seconds, local_rank, kbytes, kflops, peaks)

    # ---- GQA path on the same weights and latent (config 2: expanded cache, s_q = 2)
    w2 = synth.WORKLOADS["C2"].with_(seed=w1.seed)
    x2 = synth.make_inputs(w2)
    q2 = torch.cat([x2["q_c"], x2["q_r"]], -1).contiguous().to(dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dec.expand_cache()  # first call also loads the kernel; the second is timed
    torch.cuda.synchronize()
    ev0.record()
    B.gqla_expand_cache(dec.dims, dec.cache, dec.w_uk, dec.w_uv, dec.k_c, dec.v, None)
    ev1.record()
    torch.cuda.synchronize()
    expand_ms = ev0.elapsed_time(ev1)
    kern_g = B.kernel_for(dec.dims, torch.bfloat16, w2.s_q, "gqa")
    # balanced plan (negative split count = slots per sequence) unless a fixed split count is forced
    W_g = B.gqla_balanced_workers(dec.dims, torch.bfloat16, w2.s_q, "gqa")
    if args.splits != 0:
        S_g = args.splits
    elif W_g > 0 and args.plan != "fixed":
        S_g = -2
    else:
        S_g = pick_splits(w2.batch, w2.g, w2.seqlen, n_sm)
    if S_g < 0:
        plan_g, _ = B.gqla_balanced_plan([int(t) for t in x["seqlens"]], -S_g, W_g)
        pieces_g = sum(1 for pl in plan_g for lo, hi in pl if hi > lo) / w2.batch
    else:
        pieces_g = S_g
    og_part = dec._get("o_part_g", (w2.batch, abs(S_g), w2.s_q, w2.h_q, w2.d_h), torch.float32)
    lg_part = dec._get("lse_part_g", (w2.batch, abs(S_g), w2.s_q, w2.h_q), torch.float32)
    og = dec._get("o_g", (w2.batch, w2.s_q, w2.h_q, w2.d_h), torch.bfloat16)
    gev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    it["i"] = 0

    def gqa_step_instrumented():
        a, b = gev[it["i"]]
        it["i"] += 1
        a.record()
        B.gqla_decode_gqa(dec.dims, q2, dec.k_c, dec.v, dec.k_r, dec.seq_start, dec.seqlens, dec.scale, S_g, og_part,
                          lg_part, dec.status)
        b.record()
        B.gqla_combine_splits(og_part, lg_part, og, None)

    for _ in range(warmup):
        dec.gqa_step(q2, S_g)
    replay_gqa, _ = dec.capture(dec.gqa_step, q2, S_g)
    for _ in range(warmup):
        replay_gqa()
    gqa_ms = time_region(replay_gqa, steps, dist_on) / steps
    gqa_eager_ms = time_region(gqa_step_instrumented, steps, dist_on) / steps
    dec.check_status()
    gk_eager_ms = statistics.mean(a.elapsed_time(b) for a, b in gev)
    # The events of the eager pass cut the kernel off from its neighbours (no overlap of its set-up with the
    # previous kernel's tail), which costs this kernel more than the absorb one: its roofline figure comes from
    # the kernel running back to back.
    gk_ms = kernel_ms_back_to_back(
        lambda: B.gqla_decode_gqa(dec.dims, q2, dec.k_c, dec.v, dec.k_r, dec.seq_start, dec.seqlens, dec.scale, S_g,
                                  og_part, lg_part, dec.status), steps)
    gbytes = acct.decode_kernel_bytes("gqa", h_q=w2.h_q, g=w2.g, d_h=w2.d_h, r_kv=w2.r_kv, d_r=w2.d_r, s_q=w2.s_q,
                                      batch=w2.batch, total_tokens=total_tokens, num_splits=pieces_g)
    gflops = acct.gqa_flops(w2.h_q, w2.d_h, w2.d_r, w2.s_q, total_tokens)
    g_gbs = gbytes / (gk_ms * 1e-3) / 1e9
    g_sustained = None
    if world == 1 and not args.no_sustained:
        g_sustained = sustained_figures(
            lambda: B.gqla_decode_gqa(dec.dims, q2, dec.k_c, dec.v, dec.k_r, dec.seq_start, dec.seqlens, dec.scale, S_g,
                                      og_part, lg_part, dec.status), args.sustained_seconds, local_rank, gbytes, gflops, peaks)
    paths = {
        "absorb": {"workload": "C1", "s_q": w1.s_q, "num_splits": S_a,
                   "plan": "balanced" if S_a < 0 else "fixed", "pieces_per_sequence": pieces_a, "kernel": kern_a, "ms_per_step": ms_per_step, "ms_per_step_eager": eager_ms,
                   "tokens_per_s": value, "decode_kernel_us": kern_ms * 1e3, "gbs": gbs, "tflops": tfs},
        "gqa": {"workload": "C2", "s_q": w2.s_q, "num_splits": S_g,
                "plan": "balanced" if S_g < 0 else "fixed", "pieces_per_sequence": pieces_g, "kernel": kern_g, "ms_per_step": gqa_ms,
                "ms_per_step_eager": gqa_eager_ms,
                "tokens_per_s": world * w2.batch * w2.s_q / (gqa_ms * 1e-3), "decode_kernel_us": gk_ms * 1e3,
                "decode_kernel_us_in_eager_chain": gk_eager_ms * 1e3,

                "gbs": g_gbs, "tflops": gflops / (gk_ms * 1e-3) / 1e12,
                "roofline": {"bound": "hbm", "achieved": g_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": g_gbs / peaks["hbm_gbs"], "frac_of_8tbs": g_gbs / 8000.0,
                             "algorithmic_bytes": gbytes, "peak_source": f"of {peak_kind}", "sustained": g_sustained},
                "expand_cache_ms_one_shot": expand_ms},
    }

    # ---- the same two workloads over an FP8 cache, then the other workloads of the metric: rank 0 at N=1 only
    # (the C3 caches take 2.5 + 9 GB)
    if world == 1 and not args.no_fp8_paths:
        paths.update(fp8_paths(dec, x, x2, q2, peaks, peak_kind, min(steps, 50)))
    if world == 1 and not args.no_extra_paths:
        del replay_e2e, replay_gqa, replay_absorb
        paths.update(extra_paths(dev, local_rank, min(steps, 30), 3, args.sustained_seconds))

    # ---- CPU baseline: the oracle as it stands, rank 0 at N=1 only
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        n_seqs = w1.batch
        passes = 20  # about 10-15 s of CPU work: one pass over the whole C1 batch takes ~0.5-0.7 s on 16 cores
        val, per_step, cores = oracle_tokens_per_s(w1, x, n_seqs, passes, 1)
        cpu = {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"all {n_seqs} sequences of C1, all heads, {passes} timed passes ({per_step:.2f} s each)"}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "C1 canonical absorb path: h_q=128 g=8 d_h=128 r_kv=512 d_r=64 B=64 T=4096 s_q=1 "
                                   "bf16 cache (576 elems/token)", "num_splits": S_a, "parallelism": "replicas only",
                       "l2": "inputs larger than L2 (302 MB cache vs 126 MB L2); no flush",
                       "launch": "one CUDA-graph replay per step (3 kernels: absorb_q, decode_absorb_final, up_proj with one piece per sequence; absorb_q, decode_absorb, combine_up_proj otherwise); kernel time from an eager pass with events"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": 3 * steps, "roofline": roof, "cpu_baseline": cpu,
            # the two targets as their statement defines them: fractions of the NOMINAL roofline
            # min(2.25 PFLOP/s, bytes / 8 TB/s), not of the peaks measured on this GPU
            "targets": {"absorb_frac_of_nominal_roofline": roof["frac_of_nominal_roofline"], "absorb_target": 0.60,
                           "gqa_frac_of_8tbs": g_gbs / 8000.0, "gqa_target": 0.75},
            "paths": paths,
        }
        print(json.dumps(line))
    if dist_on:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--splits", type=int, default=0,
                    help="force the split count of both paths (0 = automatic; negative = balanced plan with that many slots)")
    ap.add_argument("--plan", default="auto", choices=["auto", "fixed"],
                    help="auto: balanced split plan where the kernels support it; fixed: equal chunks per sequence")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the long back-to-back loops of the two decode kernels")
    ap.add_argument("--sustained-seconds", type=float, default=1.0)
    ap.add_argument("--no-extra-paths", action="store_true", help="skip the C3 / C4 entries of \"paths\"")
    ap.add_argument("--no-fp8-paths", action="store_true", help="skip the FP8-cache entries of \"paths\"")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
