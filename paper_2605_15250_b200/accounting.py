"""Algorithmic bytes / FLOPs of the two decode paths (paper Sec. 4.2) for roofline reporting.

What the method must move and compute -- never the h_q-fold MHA cache it avoids:
  absorb:  cache bytes 2 (r_kv + d_r) sum_b T_b  (read once, independent of s_q and h_q)
           FLOPs 2 sum_b T_b h_q s_q (2 r_kv + d_r)
  GQA:     cache bytes 2 (2 g d_h + d_r) sum_b T_b  (k^R counted once)
           FLOPs 2 sum_b T_b h_q s_q (2 d_h + d_r)
plus the query, output and split-partial traffic of the kernel itself.
"""
from __future__ import annotations


def absorb_cache_bytes(r_kv: int, d_r: int, total_tokens: int, elem: int = 2) -> int:
    return elem * (r_kv + d_r) * total_tokens


def gqa_cache_bytes(g: int, d_h: int, d_r: int, total_tokens: int, elem: int = 2) -> int:
    return elem * (2 * g * d_h + d_r) * total_tokens


def absorb_flops(h_q: int, r_kv: int, d_r: int, s_q: int, total_tokens: int) -> int:
    return 2 * total_tokens * h_q * s_q * (2 * r_kv + d_r)


def gqa_flops(h_q: int, d_h: int, d_r: int, s_q: int, total_tokens: int) -> int:
    return 2 * total_tokens * h_q * s_q * (2 * d_h + d_r)


def decode_kernel_bytes(path: str, *, h_q: int, g: int, d_h: int, r_kv: int, d_r: int, s_q: int, batch: int,
                        total_tokens: int, num_splits: float, elem: int = 2, final: bool = False) -> int:
    """Algorithmic bytes of ONE decode-kernel launch: cache once + queries + fp32 partials and LSE.
    num_splits = partials written per sequence (under the balanced plan: live pieces / batch).
    final: the whole-sequence absorb call, which writes the output once in the storage type and no LSE."""
    rows = batch * s_q * h_q
    if path == "absorb":
        cache = absorb_cache_bytes(r_kv, d_r, total_tokens, elem)
        q = elem * rows * (r_kv + d_r)
        part = elem * rows * r_kv if final else 4 * rows * num_splits * (r_kv + 1)
    else:
        cache = gqa_cache_bytes(g, d_h, d_r, total_tokens, elem)
        q = elem * rows * (d_h + d_r)
        part = 4 * rows * num_splits * (d_h + 1)
    return int(cache + q + part)


def roofline_time(flops: float, nbytes: float, peak_flops: float, bw: float) -> float:
    """max(F / FLOPs_max, B / BW): the step time of the paper's Table "roofline"."""
    return max(flops / peak_flops, nbytes / bw)
