"""Seeded synthetic inputs for the GQLA decode workloads.

This module holds no attention arithmetic: it only names the workload shapes
and draws random tensors.  Both the CUDA binding's callers and the CPU checker
take their inputs from here so that they see identical bits.

Shapes follow the paper's canonical tuple (h_q, g, d_h, d_h^R, r_kv) =
(128, 8, 128, 64, 512) of Sec. 4.2 and its LLaMA-3-8B conversion shape
(h_q=32, g=8, d_h=128 -> r_kv=512, d_h^R=64) of Sec. 5.  The paper's workloads
need no dataset, only shapes; values are i.i.d. normal:
activations q^C, q^R, c^KV, k^R ~ N(0, 1) and up-projections
W^UK, W^UV ~ N(0, 1)/sqrt(r_kv), which makes the scaled scores unit variance.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    h_q: int
    g: int
    d_h: int
    r_kv: int
    d_r: int
    batch: int
    s_q: int
    dtype: str  # "bf16" or "f32": storage type of every tensor
    seed: int
    seqlen: int = 0  # fixed length, or
    seqlen_range: tuple[int, int] | None = None  # inclusive uniform range
    d_v: int = 0  # value head dim d_h^V of the MLA -> GQLA factorisation (Sec. 3.2); 0 = d_h (Sec. 3.1)

    @property
    def dv(self) -> int:
        return self.d_v if self.d_v > 0 else self.d_h

    @property
    def scale(self) -> float:
        """Softmax scale 1/sqrt(d_h + d_h^R) of Eqs. (mha)/(mqa)."""
        return 1.0 / float(np.sqrt(self.d_h + self.d_r))

    @property
    def d_abs(self) -> int:
        return self.r_kv + self.d_r

    @property
    def d_gqa(self) -> int:
        return self.d_h + self.d_r

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS = {
    # tiny oracle check
    "C0": Workload("C0", 8, 2, 16, 32, 8, batch=1, s_q=1, dtype="f32", seed=0xC0, seqlen=64),
    # canonical absorb path
    "C1": Workload("C1", 128, 8, 128, 512, 64, batch=64, s_q=1, dtype="bf16", seed=0xC1, seqlen=4096),
    # canonical GQA path with MTP: same weights and latent as C1 (same seed), s_q = 2
    "C2": Workload("C2", 128, 8, 128, 512, 64, batch=64, s_q=2, dtype="bf16", seed=0xC1, seqlen=4096),
    # LLaMA-3-8B-shaped, ragged
    "C3": Workload("C3", 32, 8, 128, 512, 64, batch=128, s_q=1, dtype="bf16", seed=0xC3,
                   seqlen_range=(512, 32768)),
    # long-context split-KV stress
    "C4": Workload("C4", 128, 8, 128, 512, 64, batch=4, s_q=1, dtype="bf16", seed=0xC4, seqlen=131072),
}

# tensor ids: one independent Philox stream per tensor of a workload
_T_SEQLENS, _T_QC, _T_QR, _T_WUK, _T_WUV, _T_CACHE = range(6)
_CHUNK = 1 << 24


def _rng(seed: int, tensor_id: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, tensor_id]))


def _torch_dtype(dtype: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]


def _normal(seed: int, tensor_id: int, shape, dtype: str, mul: float = 1.0) -> torch.Tensor:
    """N(0,1)*mul drawn in fp32, rounded (nearest-even) to the storage dtype."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=_torch_dtype(dtype))
    rng = _rng(seed, tensor_id)
    for lo in range(0, n, _CHUNK):
        m = min(_CHUNK, n - lo)
        x = rng.standard_normal(m, dtype=np.float32)
        if mul != 1.0:
            x *= np.float32(mul)
        out[lo:lo + m] = torch.from_numpy(x).to(out.dtype)
    return out.view(*shape)


def make_seqlens(w: Workload) -> np.ndarray:
    """int32 [batch] cache lengths (each counts the step's s_q new tokens)."""
    if w.seqlen_range is not None:
        lo, hi = w.seqlen_range
        return _rng(w.seed, _T_SEQLENS).integers(lo, hi + 1, size=w.batch).astype(np.int32)
    return np.full((w.batch,), w.seqlen, dtype=np.int32)


def make_inputs(w: Workload, seqlens: np.ndarray | None = None, q_gain: float = 1.0,
                cache_device: torch.device | str | None = None) -> dict:
    """CPU tensors of one decode step.

    cache_device: draw the cache (by far the largest tensor) on that device with torch's seeded
    generator instead of on the CPU -- same distribution, different bits; for timing runs of the
    multi-gigabyte workloads, never for a comparison with the CPU checker.

    q_gain multiplies both query parts: 1.0 gives unit-variance scores (flat
    softmax, outputs ~1/sqrt(T)); 4.0 gives a peaked softmax whose outputs are
    O(1), which is the more discriminating parity case.

    Returns q_c [B,s_q,h_q,d_h], q_r [B,s_q,h_q,d_r], w_uk [g,r_kv,d_h], w_uv [g,r_kv,d_v],
    cache [N, r_kv+d_r] (sequence b owns rows seq_start[b] .. +seqlens[b]),
    seq_start int64 [B], seqlens int32 [B].
    """
    if seqlens is None:
        seqlens = make_seqlens(w)
    seqlens = np.asarray(seqlens, dtype=np.int32)
    assert seqlens.shape == (w.batch,)
    seq_start = np.zeros((w.batch,), dtype=np.int64)
    seq_start[1:] = np.cumsum(seqlens.astype(np.int64))[:-1]
    n_rows = int(seqlens.astype(np.int64).sum())
    B, s, h = w.batch, w.s_q, w.h_q
    if cache_device is not None:
        gen = torch.Generator(device=cache_device)
        gen.manual_seed(w.seed)
        cache = torch.empty((max(n_rows, 1), w.d_abs), dtype=_torch_dtype(w.dtype), device=cache_device)
        step = 1 << 18
        for lo in range(0, cache.shape[0], step):
            hi = min(lo + step, cache.shape[0])
            cache[lo:hi] = torch.randn((hi - lo, w.d_abs), generator=gen, device=cache_device, dtype=torch.float32)
        cache = cache[:n_rows]
    else:
        cache = _normal(w.seed, _T_CACHE, (max(n_rows, 1), w.d_abs), w.dtype)[:n_rows]
    return {
        "q_c": _normal(w.seed, _T_QC, (B, s, h, w.d_h), w.dtype, q_gain),
        "q_r": _normal(w.seed, _T_QR, (B, s, h, w.d_r), w.dtype, q_gain),
        "w_uk": _normal(w.seed, _T_WUK, (w.g, w.r_kv, w.d_h), w.dtype, 1.0 / float(np.sqrt(w.r_kv))),
        "w_uv": _normal(w.seed, _T_WUV, (w.g, w.r_kv, w.dv), w.dtype, 1.0 / float(np.sqrt(w.r_kv))),
        "cache": cache,
        "seq_start": torch.from_numpy(seq_start),
        "seqlens": torch.from_numpy(seqlens.copy()),
    }


def make_queries(w: Workload, q_gain: float = 1.0) -> dict:
    """The two query tensors of make_inputs alone (same streams, same bits)."""
    B, s, h = w.batch, w.s_q, w.h_q
    return {"q_c": _normal(w.seed, _T_QC, (B, s, h, w.d_h), w.dtype, q_gain),
            "q_r": _normal(w.seed, _T_QR, (B, s, h, w.d_r), w.dtype, q_gain)}


def to_paged(t: torch.Tensor, seq_start, seqlens, page_size: int, seed: int, fill: float = 3.0, spare_pages: int = 3):
    """Scatters packed rows [N, ...] into a paged layout: the pages of every sequence are placed at seeded
    random positions of a pool with a few spare pages; rows no sequence owns hold `fill` (finite, so a
    tile that reads past a sequence's end sees harmless values).  Returns (paged [n_pages * page_size, ...],
    block_table int32 [B, max_pages]); unused table entries are -1 ... never read."""
    seqlens = np.asarray(seqlens)
    pages_of = [(int(T) + page_size - 1) // page_size for T in seqlens]
    max_pages = max(1, max(pages_of) if len(pages_of) else 1)
    n_pages = sum(pages_of) + spare_pages
    order = _rng(seed, 99).permutation(n_pages)
    paged = torch.full((n_pages * page_size, *t.shape[1:]), fill, dtype=t.dtype)
    table = np.full((len(seqlens), max_pages), -1, dtype=np.int32)
    nxt = 0
    for b, T in enumerate(seqlens):
        for k in range(pages_of[b]):
            page = int(order[nxt]); nxt += 1
            table[b, k] = page
            lo = k * page_size
            n = min(page_size, int(T) - lo)
            src = int(seq_start[b]) + lo
            paged[page * page_size:page * page_size + n] = t[src:src + n]
    return paged, torch.from_numpy(table)


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a stored tensor to float64 (for the CPU checker)."""
    return t.detach().cpu().to(torch.float64).numpy()
