"""Device-side timing helpers shared by bench.py and the sweep."""
from __future__ import annotations

import statistics
import subprocess
import time

import torch


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a timed region runs (reads only)."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "20", "-i", str(self.index)], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        self.proc.terminate()
        out, _ = self.proc.communicate(timeout=10)
        sm, mx, pw, reasons = [], [], [], set()
        for line in out.strip().splitlines():
            f = [c.strip() for c in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def kernel_ms_back_to_back(launch, launches: int) -> float:
    """Mean device time of one launch when the kernel runs back to back: `launches` launches replayed from CUDA
    graphs of ten (so the host's launch cost cannot stretch the figure), one event pair around all of them."""
    per_graph = 10
    launch()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(per_graph):
                launch()
    torch.cuda.current_stream().wait_stream(side)
    replays = max(1, launches // per_graph)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (replays * per_graph)


def kernel_sustained(launch, seconds: float, gpu_index: int) -> dict:
    """The kernel running back to back for at least `seconds` (graphs of ten launches), with the SM clock
    sampled meanwhile: mean device time per launch, the median clock, and their product in cycles (which
    compares across GPUs of a pool whose power-capped clocks differ)."""
    per_graph = 10
    launch()
    g = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            for _ in range(per_graph):
                launch()
    torch.cuda.current_stream().wait_stream(side)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g.replay()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(3):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    est_ms = max(e0.elapsed_time(e1) / 3, 1e-3)
    replays = max(3, int(seconds * 1e3 / est_ms) + 1)
    sampler = ClockSampler(gpu_index)
    sampler.start()
    time.sleep(0.05)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    us = e0.elapsed_time(e1) * 1e3 / (replays * per_graph)
    mhz = clocks.get("sm_mhz")
    return {"kernel_us": us, "launches": replays * per_graph, "loop_s": e0.elapsed_time(e1) * 1e-3, "sm_mhz": mhz,
            "kernel_cycles": us * mhz if mhz else None, "power_w": clocks.get("power_w"), "reasons": clocks.get("reasons")}
