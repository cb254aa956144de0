"""How fast can the absorb kernel's K stream be fed?  (python -m paper_2605_15250_b200.stream_probe)

128 (or 148) CTAs pull the [64 rows x 64 columns] TMA boxes of a bf16 latent cache through a ring of three-box
groups, as the decode kernel's K producer does, and nothing consumes them.  Printed per ring depth: time for the
C1-sized cache (64 sequences x 4096 rows), TB/s, and the same with every tile re-reading L2-resident rows.  The
one-group ring gives the round-trip time of a group (request -> landed -> slot handed back -> next request).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import torch

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(PKG_DIR, "libgqla_probe.so")
SRC = os.path.join(PKG_DIR, "csrc", "stream_probe.cu")


def build() -> str:
    if not os.path.exists(LIB) or os.path.getmtime(LIB) < max(os.path.getmtime(SRC), os.path.getmtime(
            os.path.join(PKG_DIR, "csrc", "tc_common.cuh"))):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "--expt-relaxed-constexpr",
               "-shared", "-Xcompiler", "-fPIC", "-cudart", "static", "-o", LIB, SRC]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return LIB


def main() -> None:
    lib = ctypes.CDLL(build())
    lib.gqla_stream_probe.restype = ctypes.c_int
    lib.gqla_stream_probe.argtypes = [ctypes.c_void_p, ctypes.c_longlong, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    assert torch.cuda.is_available(), "the probe needs a CUDA device"
    seqs, T, tiles = 74, 4096, 32
    cache = torch.randn((seqs * T, 576), device="cuda").to(torch.bfloat16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    st = torch.cuda.current_stream().cuda_stream

    def run(n_ctas: int, depth: int, l2: int, reps: int = 20) -> float:
        call = lambda: lib.gqla_stream_probe(cache.data_ptr(), seqs * T, n_ctas, tiles, T, depth, l2, status.data_ptr(), st)
        for _ in range(3):
            assert call() == 0
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / reps

    for n_ctas in (128, 148):
        for depth in (1, 2, 3, 4, 6, 9):
            nbytes = n_ctas * tiles * 9 * 8192
            us, us_l2 = run(n_ctas, depth, 0), run(n_ctas, depth, 1)
            trip = f"   round trip of a group {us / (tiles * 3):4.2f} / {us_l2 / (tiles * 3):4.2f} us" if depth == 1 else ""
            print(f"ctas {n_ctas} ring {depth} groups ({depth * 24} KB in flight per CTA): HBM {us:6.1f} us {nbytes / us / 1e6:5.2f} TB/s"
                  f"   L2-resident {us_l2:6.1f} us {nbytes / us_l2 / 1e6:5.2f} TB/s{trip}", flush=True)
    assert int(status.item()) == 0, "a bounded wait expired"


if __name__ == "__main__":
    main()
