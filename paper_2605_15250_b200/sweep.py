"""Timing sweep of both decode paths over the five workloads (python -m paper_2605_15250_b200.sweep).

For every (workload, path, s_q, split plan) it times the decode kernel alone (running back to back, replayed
from CUDA graphs of ten launches) and the whole path chain as one CUDA-graph replay per step, and prints one
JSON line with tokens/s, algorithmic GB/s and TFLOP/s, and the fraction of the roofline time max(bytes/BW, FLOPs/peak)
against the measured peaks (MEASURED_PEAKS.json beside bench.py, if present) and the nominal B200
figures (8 TB/s, 2.25 PFLOP/s dense bf16).  Inputs are the seeded synthetic workloads of synth.py.
"""
from __future__ import annotations

import argparse
import json
import os

import torch

from . import accounting as acct
from . import binding as B
from . import build as gbuild
from . import synth
from .decoder import GqlaDecoder
from .timing import kernel_ms_back_to_back

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            return json.load(fh), "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0}, "fallback"


def _pieces(seqlens, S: int, W: int, batch: int) -> float:
    if S > 0:
        return float(S)
    plan, _ = B.gqla_balanced_plan([int(t) for t in seqlens], -S, W)
    return sum(1 for pl in plan for lo, hi in pl if hi > lo) / batch


def time_paged(dec: GqlaDecoder, w: synth.Workload, x: dict, path: str, S: int, page_size: int, steps: int,
               warmup: int) -> dict:
    """The decode kernel alone over a pool of shuffled pages holding the same rows (kernel time only)."""
    dev = dec.device
    slots = abs(S)
    total_tokens = int(x["seqlens"].sum())
    cache_p, table = synth.to_paged(x["cache"], x["seq_start"], x["seqlens"].numpy(), page_size, seed=w.seed + 1)
    cache_p, table = cache_p.to(dev), table.to(dev)
    if path == "absorb":
        q_hat = torch.randn((w.batch, w.s_q, w.h_q, w.d_abs), device=dev).to(torch.bfloat16)
        o_part = torch.empty((w.batch, slots, w.s_q, w.h_q, w.r_kv), dtype=torch.float32, device=dev)
        lse_part = torch.empty((w.batch, slots, w.s_q, w.h_q), dtype=torch.float32, device=dev)

        def kernel():
            B.gqla_decode_absorb_paged(dec.dims, q_hat, cache_p, table, page_size, dec.seqlens, dec.scale, S, o_part,
                                       lse_part, dec.status)
    else:
        k_c = torch.empty((cache_p.shape[0], w.g, w.d_h), dtype=torch.bfloat16, device=dev)
        v = torch.empty_like(k_c)
        B.gqla_expand_cache(dec.dims, cache_p, dec.w_uk, dec.w_uv, k_c, v, None)
        q = torch.randn((w.batch, w.s_q, w.h_q, w.d_gqa), device=dev).to(torch.bfloat16)
        o_part = torch.empty((w.batch, slots, w.s_q, w.h_q, w.d_h), dtype=torch.float32, device=dev)
        lse_part = torch.empty((w.batch, slots, w.s_q, w.h_q), dtype=torch.float32, device=dev)

        def kernel():
            B.gqla_decode_gqa_paged(dec.dims, q, k_c, v, cache_p[:, w.r_kv:], table, page_size, dec.seqlens, dec.scale, S,
                                    o_part, lse_part, dec.status)
    for _ in range(warmup):
        kernel()
    k_us = kernel_ms_back_to_back(kernel, steps) * 1e3
    dec.check_status()
    return {"workload": w.name, "path": path, "s_q": w.s_q, "batch": w.batch, "total_tokens": total_tokens,
            "layout": f"paged, {page_size} rows per page, shuffled", "plan": "balanced" if S < 0 else "fixed",
            "slots": slots, "kernel_us": round(k_us, 1)}


def time_case(dec: GqlaDecoder, w: synth.Workload, x: dict, path: str, S: int, steps: int, warmup: int) -> dict:
    dev = dec.device
    total_tokens = int(x["seqlens"].sum())
    slots = abs(S)
    if path == "absorb":
        q_c, q_r = x["q_c"].to(dev), x["q_r"].to(dev)
        args = (q_c, q_r, S)
        step = dec.absorb_step
        q_hat = dec._get("q_hat", (w.batch, w.s_q, w.h_q, w.d_abs), torch.bfloat16)
        o_part = dec._get("o_part_a", (w.batch, slots, w.s_q, w.h_q, w.r_kv), torch.float32)
        lse_part = dec._get("lse_part_a", (w.batch, slots, w.s_q, w.h_q), torch.float32)

        o_hat = dec._get("o_hat", (w.batch, w.s_q, w.h_q, w.r_kv), torch.bfloat16)

        def kernel():
            if S == 1:  # the call the chain uses with one piece per sequence
                B.gqla_decode_absorb_final(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, o_hat, None,
                                           dec.status)
            else:
                B.gqla_decode_absorb(dec.dims, q_hat, dec.cache, dec.seq_start, dec.seqlens, dec.scale, S, o_part,
                                     lse_part, dec.status)

        flops = acct.absorb_flops(w.h_q, w.r_kv, w.d_r, w.s_q, total_tokens)
    else:
        q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().to(dev)
        args = (q, S)
        step = dec.gqa_step
        o_part = dec._get("o_part_g", (w.batch, slots, w.s_q, w.h_q, w.d_h), torch.float32)
        lse_part = dec._get("lse_part_g", (w.batch, slots, w.s_q, w.h_q), torch.float32)

        def kernel():
            B.gqla_decode_gqa(dec.dims, q, dec.k_c, dec.v, dec.k_r, dec.seq_start, dec.seqlens, dec.scale, S, o_part,
                              lse_part, dec.status)

        flops = acct.gqa_flops(w.h_q, w.d_h, w.d_r, w.s_q, total_tokens)
    W = B.gqla_balanced_workers(dec.dims, torch.bfloat16, w.s_q, path)
    if S < 0 and W <= 0:
        return {}
    pieces = _pieces(x["seqlens"], S, W, w.batch)
    nbytes = acct.decode_kernel_bytes(path, h_q=w.h_q, g=w.g, d_h=w.d_h, r_kv=w.r_kv, d_r=w.d_r, s_q=w.s_q,
                                      batch=w.batch, total_tokens=total_tokens, num_splits=pieces,
                                      final=path == "absorb" and S == 1)
    replay, _ = dec.capture(step, *args)
    for _ in range(warmup):
        replay()
        kernel()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        replay()
    e1.record()
    torch.cuda.synchronize()
    chain_us = e0.elapsed_time(e1) * 1e3 / steps
    k_us = kernel_ms_back_to_back(kernel, steps) * 1e3
    dec.check_status()
    peaks, kind = _peaks()
    t = k_us * 1e-6
    out = {
        "workload": w.name, "path": path, "s_q": w.s_q, "batch": w.batch, "total_tokens": total_tokens,
        "plan": "balanced" if S < 0 else "fixed", "slots": slots, "pieces_per_sequence": round(pieces, 3),
        "kernel": B.kernel_for(dec.dims, torch.bfloat16, w.s_q, path), "kernel_us": round(k_us, 1),
        "path_us": round(chain_us, 1), "tokens_per_s": round(w.batch * w.s_q / (chain_us * 1e-6)),
        "gbs": round(nbytes / t / 1e9, 1), "tflops": round(flops / t / 1e12, 1),
        f"frac_of_{kind}_roofline": round(acct.roofline_time(flops, nbytes, peaks["bf16_tflops"] * 1e12,
                                                              peaks["hbm_gbs"] * 1e9) / t, 3),
        "frac_of_nominal_roofline": round(acct.roofline_time(flops, nbytes, NOMINAL["bf16_tflops"] * 1e12,
                                                              NOMINAL["hbm_gbs"] * 1e9) / t, 3),
        "intensity_flop_per_byte": round(flops / nbytes, 1),
    }
    return out


def run(names, steps: int, warmup: int, paths=("absorb", "gqa")):
    gbuild.build()
    B.lib()
    assert torch.cuda.is_available(), "the sweep needs a CUDA device"
    dev = torch.device("cuda", 0)
    cases = {
        "C1": [("absorb", 1, (1, -3))],
        "C2": [("gqa", 2, (1, -2)), ("absorb", 2, (1, -3))],
        "C3": [("absorb", 1, (4, -3)), ("absorb", 2, (4, -3)), ("gqa", 1, (4, -2)), ("gqa", 2, (4, -2))],
        "C4": [("absorb", 1, (1, 8, 32, 128, -32)), ("absorb", 2, (1, 8, 32, 128, -32)), ("gqa", 1, (1, 8, 32, 128, -32)),
               ("gqa", 2, (1, 8, 32, 128, -32))],
    }
    for name in names:
        base = synth.WORKLOADS[name]
        dec = None
        todo = [c for c in cases[name] if c[0] in paths]
        for path, s_q, plans in todo:
            w = base.with_(s_q=s_q)
            x = synth.make_inputs(w)
            if dec is None:
                dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].to(dev), x["w_uv"].to(dev),
                                  x["cache"].to(dev), x["seq_start"].to(dev), x["seqlens"].to(dev), w.scale)
                if any(p == "gqa" for p, _, _ in todo):
                    dec.expand_cache()
            for S in plans:
                res = time_case(dec, w, x, path, S, steps, warmup)
                if res:
                    print(json.dumps(res), flush=True)
            # the same kernel over a paged pool, on the two workloads the benchmark quotes
            if (name, path) in (("C1", "absorb"), ("C2", "gqa")):
                print(json.dumps(time_paged(dec, w, x, path, plans[0] if name == "C1" else plans[-1], 128, steps, warmup)),
                      flush=True)
        del dec
        torch.cuda.empty_cache()


def markdown(path: str) -> None:
    """Prints the JSON lines of an earlier run as a markdown table."""
    print("| config | path | s_q | split plan | pieces/seq | decode kernel µs | path µs | tokens/s (path) | GB/s | TFLOP/s | "
          "of measured roofline | of nominal roofline |")
    print("|---|---|---|---|---|---|---|---|---|---|---|---|")
    with open(path) as fh:
        for line in fh:
            r = json.loads(line)
            if "layout" in r:
                continue
            plan = f"{r['plan']}, {'S=' if r['plan'] == 'fixed' else ''}{r['slots']}{'' if r['plan'] == 'fixed' else ' slots'}"
            meas = r.get("frac_of_measured_roofline", r.get("frac_of_fallback_roofline"))
            print(f"| {r['workload']} | {r['path']} | {r['s_q']} | {plan} | {r['pieces_per_sequence']:.2f} | {r['kernel_us']} | "
                  f"{r['path_us']} | {r['tokens_per_s']:,} | {r['gbs']:.0f} | {r['tflops']:.0f} | {meas:.3f} | "
                  f"{r['frac_of_nominal_roofline']:.3f} |")


if __name__ == "__main__":
    ap = argparse.ArgumentParser()
    ap.add_argument("--workloads", default="C1,C2,C3,C4")
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--paths", default="absorb,gqa", help="decode paths to time (the GQA path expands the cache first)")
    ap.add_argument("--markdown", default="", help="print the JSON lines of an earlier run (a file) as a markdown table and exit")
    a = ap.parse_args()
    if a.markdown:
        markdown(a.markdown)
    else:
        run(a.workloads.split(","), a.steps, a.warmup, tuple(a.paths.split(",")))
