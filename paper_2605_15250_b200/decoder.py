"""Decode-step driver: owns the device buffers of one GQLA attention layer and chains
the library calls of each path.  No arithmetic happens here -- torch only allocates."""
from __future__ import annotations

import torch

from . import binding as B


class GqlaDecoder:
    """One layer's decode attention over a resident KV cache, through either path.

    Absorb path (Eq. (mqa)):  absorb_q -> decode_absorb -> combine_splits -> up_proj
    GQA path    (Eq. (mha)):  decode_gqa -> combine_splits   (after a one-shot expand_cache)
    """

    def __init__(self, h_q: int, g: int, d_h: int, r_kv: int, d_r: int, w_uk: torch.Tensor, w_uv: torch.Tensor,
                 cache: torch.Tensor, seq_start: torch.Tensor | None, seqlens: torch.Tensor, scale: float,
                 block_table: torch.Tensor | None = None, page_size: int = 0):
        """Packed cache: `seq_start` [B] int64.  Paged cache: `block_table` [B, max_pages] int32 of page numbers
        and `page_size` rows per page (`seq_start` is then ignored and may be None)."""
        assert cache.is_cuda and w_uk.is_cuda and w_uv.is_cuda
        assert (block_table is None) == (page_size == 0) and (block_table is not None or seq_start is not None)
        self.block_table, self.page_size = block_table, int(page_size)
        self.dims = B.make_dims(h_q, g, d_h, r_kv, d_r)
        self.h_q, self.g, self.d_h, self.r_kv, self.d_r = h_q, g, d_h, r_kv, d_r
        self.w_uk, self.w_uv, self.cache = w_uk, w_uv, cache
        self.seq_start, self.seqlens = seq_start, seqlens
        self.scale = float(scale)
        self.dtype = cache.dtype
        self.device = cache.device
        self.batch = int(seqlens.shape[0])
        self.k_c = self.v = self.k_r = None
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self._buf = {}

    def _get(self, name: str, shape, dtype) -> torch.Tensor:
        key = (name, tuple(shape), dtype)
        t = self._buf.get(key)
        if t is None:
            t = torch.empty(shape, dtype=dtype, device=self.device)
            self._buf[key] = t
        return t

    # ---- one-shot cache expansion (Sec. 3.1) ----
    def expand_cache(self, alias_k_r: bool = True) -> None:
        """Builds K_C, V [N,g,d_h].  With alias_k_r the shared RoPE key is read in place from
        the latent cache's last d_r columns (the paper's "no-op view"); otherwise it is copied."""
        N = self.cache.shape[0]
        self.k_c = torch.empty((N, self.g, self.d_h), dtype=self.dtype, device=self.device)
        self.v = torch.empty((N, self.g, self.d_h), dtype=self.dtype, device=self.device)
        if alias_k_r:
            B.gqla_expand_cache(self.dims, self.cache, self.w_uk, self.w_uv, self.k_c, self.v, None)
            self.k_r = self.cache[:, self.r_kv:]
        else:
            self.k_r = torch.empty((N, self.d_r), dtype=self.dtype, device=self.device)
            B.gqla_expand_cache(self.dims, self.cache, self.w_uk, self.w_uv, self.k_c, self.v, self.k_r)

    def append_expand(self, s_q: int) -> None:
        """After a step has written s_q new latent rows per sequence (and raised seqlens): expands just
        those rows into K_C, V (and k_R unless it aliases the latent cache)."""
        if self.block_table is not None:
            raise B.GqlaError("append_expand takes the packed layout; expand the touched pages with gqla_expand_cache")
        alias = self.k_r.data_ptr() == self.cache[:, self.r_kv:].data_ptr()
        B.gqla_append_expand(self.dims, s_q, self.cache, self.seq_start, self.seqlens, self.w_uk, self.w_uv, self.k_c,
                             self.v, None if alias else self.k_r)

    # ---- absorb path ----
    def absorb_step(self, q_c: torch.Tensor, q_r: torch.Tensor, num_splits: int = 1, want_lse: bool = False,
                    fused_tail: bool = True):
        """absorb_q -> decode_absorb -> combine_up_proj (or combine_splits -> up_proj when fused_tail is off);
        with one split per sequence: absorb_q -> decode_absorb_final -> up_proj."""
        Bn, s_q = q_c.shape[0], q_c.shape[1]
        slots = abs(num_splits)  # num_splits < 0: balanced plan with that many slots per sequence
        q_hat = self._get("q_hat", (Bn, s_q, self.h_q, self.r_kv + self.d_r), self.dtype)
        o_part = self._get("o_part_a", (Bn, slots, s_q, self.h_q, self.r_kv), torch.float32)
        lse_part = self._get("lse_part_a", (Bn, slots, s_q, self.h_q), torch.float32)
        o_hat = self._get("o_hat", (Bn, s_q, self.h_q, self.r_kv), self.dtype)
        lse = self._get("lse_a", (Bn, s_q, self.h_q), torch.float32) if want_lse else None
        o = self._get("o_a", (Bn, s_q, self.h_q, self.d_h), self.dtype)
        B.gqla_absorb_q(self.dims, q_c, q_r, self.w_uk, q_hat)
        if num_splits == 1 and self.block_table is None:
            # one piece per sequence: no partials, the latent output goes straight to the up-projection
            B.gqla_decode_absorb_final(self.dims, q_hat, self.cache, self.seq_start, self.seqlens, self.scale, o_hat, lse,
                                       self.status)
            B.gqla_up_proj(self.dims, o_hat, self.w_uv, o)
            return (o, lse) if want_lse else o
        if self.block_table is None:
            B.gqla_decode_absorb(self.dims, q_hat, self.cache, self.seq_start, self.seqlens, self.scale, num_splits,
                                 o_part, lse_part, self.status)
        else:
            B.gqla_decode_absorb_paged(self.dims, q_hat, self.cache, self.block_table, self.page_size, self.seqlens,
                                       self.scale, num_splits, o_part, lse_part, self.status)
        # with many slots per sequence the fused kernel (64 rows per CTA, one slot after the other) runs out of
        # parallelism; the separate merge streams the partials with every thread of the GPU
        if fused_tail and slots <= 4:
            B.gqla_combine_up_proj(self.dims, o_part, lse_part, self.w_uv, o, lse)
        else:
            B.gqla_combine_splits(o_part, lse_part, o_hat, lse)
            B.gqla_up_proj(self.dims, o_hat, self.w_uv, o)
        return (o, lse) if want_lse else o

    # ---- GQA path ----
    def gqa_step(self, q: torch.Tensor, num_splits: int = 1, want_lse: bool = False):
        """q is [B, s_q, h_q, d_h+d_r] = [q^C ; q^R]."""
        if self.k_c is None:
            raise B.GqlaError("expand_cache() must run before the GQA path")
        Bn, s_q = q.shape[0], q.shape[1]
        slots = abs(num_splits)
        o_part = self._get("o_part_g", (Bn, slots, s_q, self.h_q, self.d_h), torch.float32)
        lse_part = self._get("lse_part_g", (Bn, slots, s_q, self.h_q), torch.float32)
        lse = self._get("lse_g", (Bn, s_q, self.h_q), torch.float32) if want_lse else None
        o = self._get("o_g", (Bn, s_q, self.h_q, self.d_h), self.dtype)
        if self.block_table is None:
            B.gqla_decode_gqa(self.dims, q, self.k_c, self.v, self.k_r, self.seq_start, self.seqlens, self.scale,
                              num_splits, o_part, lse_part, self.status)
        else:
            B.gqla_decode_gqa_paged(self.dims, q, self.k_c, self.v, self.k_r, self.block_table, self.page_size,
                                    self.seqlens, self.scale, num_splits, o_part, lse_part, self.status)
        B.gqla_combine_splits(o_part, lse_part, o, lse)
        return (o, lse) if want_lse else o

    # ---- CUDA graphs: one replay per decode step instead of four (two) host-side launches ----
    def capture(self, step, *args, warmup: int = 2):
        """Captures one call of `step` (absorb_step or gqa_step) with these argument tensors into a CUDA
        graph and returns (replay, output).  The step reads its inputs from the SAME tensors on every
        replay (copy new queries into them first) and writes the same output tensors.  All buffers are
        allocated during the warm-up calls, so nothing is allocated while capturing."""
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(warmup):
                out = step(*args)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize(self.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            out = step(*args)
        return graph.replay, out

    def check_status(self) -> None:
        """Synchronises and raises if a bounded device wait expired in any earlier call."""
        code = int(self.status.item())
        if code != 0:
            raise B.GqlaError(f"device status word = {code} (a bounded wait expired)")
