"""ctypes binding of libgqla.so: one Python function per C entry point, same names.

Argument marshalling only -- every step of the decode path runs in the CUDA
library.  torch supplies device memory and the current stream.  There is no
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_float, c_int32, c_int64, c_void_p

import torch

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
# GQLA_LIB_PATH selects another build of the same library (e.g. the -DGQLA_DEBUG one, libgqla_debug.so)
LIB_PATH = os.environ.get("GQLA_LIB_PATH") or os.path.join(_PKG_DIR, "libgqla.so")

GQLA_BF16, GQLA_F32 = 0, 1
POLICY_AUTO, POLICY_GENERIC = 0, 1


class GqlaDims(ctypes.Structure):
    """(h_q, g, d_h, r_kv, d_h^R) of the paper's Sec. 4.2."""

    _fields_ = [("h_q", c_int32), ("g", c_int32), ("d_h", c_int32), ("r_kv", c_int32), ("d_r", c_int32)]


class GqlaError(RuntimeError):
    pass


_lib = None

_PROTOTYPES = {
    "gqla_set_policy": (None, [c_int32]),
    "gqla_get_policy": (c_int32, []),
    "gqla_set_status_word": (None, [c_void_p]),
    "gqla_get_status_word": (c_void_p, []),
    "gqla_absorb_q": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_decode_absorb": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p,
                                     c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_decode_absorb_final": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p, c_int64,
                                           c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_decode_absorb_paged": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p,
                                           c_int64, c_int64, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                           c_void_p, c_void_p]),
    "gqla_decode_gqa_paged": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p,
                                        c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_int32, c_int32, c_void_p,
                                        c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_append_expand": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_int64, c_void_p, c_void_p, c_void_p,
                                     c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_expand_cache": (c_int32, [c_void_p, c_int32, c_int64, c_void_p, c_int64, c_void_p, c_void_p, c_void_p,
                                    c_void_p, c_void_p, c_void_p]),
    "gqla_decode_gqa": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p,
                                  c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                  c_void_p, c_void_p]),
    "gqla_decode_gqa_noalloc": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p,
                                          c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                          c_void_p, c_void_p]),
    "gqla_combine_splits": (c_int32, [c_int32, c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_void_p]),
    "gqla_combine_up_proj": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p,
                                       c_void_p, c_void_p, c_void_p]),
    "gqla_up_proj": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_up_proj_dv": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_expand_cache_dv": (c_int32, [c_void_p, c_int32, c_int32, c_int64, c_void_p, c_int64, c_void_p, c_void_p,
                                       c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_decode_gqa_dv": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p,
                                     c_void_p, c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                     c_void_p, c_void_p]),
    "gqla_quantize_cols_e4m3": (c_int32, [c_int32, c_int64, c_int32, c_int32, c_float, c_float, c_void_p, c_int64, c_void_p,
                                          c_void_p]),
    "gqla_quantize_rows_e4m3": (c_int32, [c_int32, c_int64, c_int32, c_int32, c_float, c_float, c_void_p, c_void_p, c_void_p,
                                          c_void_p]),
    "gqla_decode_absorb_fp8": (c_int32, [c_void_p, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p, c_void_p, c_int64,
                                         c_int64, c_float, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_decode_absorb_fp8_final": (c_int32, [c_void_p, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p, c_int64,
                                               c_int64, c_float, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "gqla_decode_gqa_fp8": (c_int32, [c_void_p, c_int32, c_int32, c_float, c_int32, c_void_p, c_void_p, c_void_p, c_void_p,
                                      c_void_p, c_int64, c_int64, c_float, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p,
                                      c_void_p]),
    "gqla_split_plan": (c_int32, [c_int32, c_int32, c_void_p, c_void_p]),
    "gqla_visible_limit": (c_int32, [c_int32, c_int32, c_int32]),
    "gqla_balanced_plan": (c_int32, [c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p]),
    "gqla_balanced_workers": (c_int32, [c_void_p, c_int32, c_int32, c_int32]),
    "gqla_group_of_head": (c_int32, [c_void_p, c_int32]),
    "gqla_kernel_for": (c_char_p, [c_void_p, c_int32, c_int32, c_int32]),
    "gqla_status_str": (c_char_p, [c_int32]),
}


def lib() -> ctypes.CDLL:
    """Loads libgqla.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise GqlaError(f"{LIB_PATH} not found: build it with `python -m paper_2605_15250_b200.build`")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _PROTOTYPES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def exported_symbols() -> list[str]:
    return sorted(_PROTOTYPES)


def _check(code: int, what: str) -> None:
    if code != 0:
        raise GqlaError(f"{what}: {lib().gqla_status_str(code).decode()} (status {code})")


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return GQLA_BF16
    if t.dtype == torch.float32:
        return GQLA_F32
    raise GqlaError(f"unsupported dtype {t.dtype}")


def _ptr(t: torch.Tensor | None) -> int | None:
    if t is None:
        return None
    if not t.is_cuda:
        raise GqlaError("expected a CUDA tensor")
    return t.data_ptr()


def _contig(*ts: torch.Tensor) -> None:
    for t in ts:
        if t is not None and not t.is_contiguous():
            raise GqlaError("expected a contiguous tensor")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_dims(h_q: int, g: int, d_h: int, r_kv: int, d_r: int) -> GqlaDims:
    return GqlaDims(h_q, g, d_h, r_kv, d_r)


def set_policy(policy: int) -> None:
    lib().gqla_set_policy(policy)


def get_policy() -> int:
    return lib().gqla_get_policy()


def set_status_word(word: torch.Tensor | None) -> None:
    """Registers the device int32 that the projection calls (absorb_q, up_proj, expand_cache, append_expand,
    combine_up_proj) report an expired device-side wait in; None unregisters.  Keep the tensor alive."""
    if word is not None:
        assert word.is_cuda and word.dtype == torch.int32 and word.numel() >= 1
    lib().gqla_set_status_word(_ptr(word))


def get_status_word() -> int:
    """Address registered with set_status_word (0 = none)."""
    return int(lib().gqla_get_status_word() or 0)


def kernel_for(dims: GqlaDims, dtype: torch.dtype, s_q: int, path: str) -> str:
    code = GQLA_BF16 if dtype == torch.bfloat16 else GQLA_F32
    return lib().gqla_kernel_for(ctypes.byref(dims), code, s_q, {"absorb": 0, "gqa": 1, "projections": 2}[path]).decode()


# ------------------------------------------------------------------ the six calls


def gqla_absorb_q(dims: GqlaDims, q_c: torch.Tensor, q_r: torch.Tensor, w_uk: torch.Tensor,
                  q_hat: torch.Tensor) -> None:
    """q_hat[B,s_q,h_q,r_kv+d_r] = [(W^UK_{j(i)})^T q_c ; q_r]  (Eq. (mqa), line 2)."""
    _contig(q_c, q_r, w_uk, q_hat)
    B, s_q = q_c.shape[0], q_c.shape[1]
    _check(lib().gqla_absorb_q(ctypes.byref(dims), _dtype_code(q_c), B, s_q, _ptr(q_c), _ptr(q_r), _ptr(w_uk),
                               _ptr(q_hat), _stream()), "gqla_absorb_q")


def gqla_decode_absorb(dims: GqlaDims, q_hat: torch.Tensor, cache: torch.Tensor, seq_start: torch.Tensor,
                       seqlens: torch.Tensor, scale: float, num_splits: int, o_part: torch.Tensor,
                       lse_part: torch.Tensor, status_word: torch.Tensor | None = None) -> None:
    """Split-KV absorb-path attention (Eq. (mqa), lines 3-5).  cache is [N, r_kv+d_r] (rows may be strided)."""
    _contig(q_hat, seq_start, seqlens, o_part, lse_part)
    assert cache.dim() == 2 and cache.stride(1) == 1
    assert seq_start.dtype == torch.int64 and seqlens.dtype == torch.int32
    assert o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q_hat.shape[0], q_hat.shape[1]
    _check(lib().gqla_decode_absorb(ctypes.byref(dims), _dtype_code(q_hat), B, s_q, scale, num_splits, _ptr(q_hat),
                                    _ptr(cache), cache.stride(0), cache.shape[0], _ptr(seq_start), _ptr(seqlens), _ptr(o_part),
                                    _ptr(lse_part), _ptr(status_word), _stream()), "gqla_decode_absorb")


def gqla_expand_cache(dims: GqlaDims, cache: torch.Tensor, w_uk: torch.Tensor, w_uv: torch.Tensor,
                      k_c: torch.Tensor, v: torch.Tensor, k_r: torch.Tensor | None) -> None:
    """K_C, V [N,g,d_h] = W^UK c, W^UV c per group; k_R [N,d_r] copied (Sec. 3.1)."""
    _contig(w_uk, w_uv, k_c, v, k_r)
    assert cache.dim() == 2 and cache.stride(1) == 1
    _check(lib().gqla_expand_cache(ctypes.byref(dims), _dtype_code(cache), cache.shape[0], _ptr(cache),
                                   cache.stride(0), _ptr(w_uk), _ptr(w_uv), _ptr(k_c), _ptr(v), _ptr(k_r),
                                   _stream()), "gqla_expand_cache")


def gqla_decode_absorb_final(dims: GqlaDims, q_hat: torch.Tensor, cache: torch.Tensor, seq_start: torch.Tensor,
                             seqlens: torch.Tensor, scale: float, o_hat: torch.Tensor, lse: torch.Tensor | None,
                             status_word: torch.Tensor | None = None) -> None:
    """Whole-sequence absorb-path attention (Eq. (mqa), lines 3-5): o_hat [B,s_q,h_q,r_kv] in the storage dtype."""
    _contig(q_hat, seq_start, seqlens, o_hat, lse)
    assert cache.dim() == 2 and cache.stride(1) == 1
    assert seq_start.dtype == torch.int64 and seqlens.dtype == torch.int32 and o_hat.dtype == q_hat.dtype
    assert lse is None or lse.dtype == torch.float32
    B, s_q = q_hat.shape[0], q_hat.shape[1]
    _check(lib().gqla_decode_absorb_final(ctypes.byref(dims), _dtype_code(q_hat), B, s_q, scale, _ptr(q_hat), _ptr(cache),
                                          cache.stride(0), cache.shape[0], _ptr(seq_start), _ptr(seqlens), _ptr(o_hat),
                                          _ptr(lse), _ptr(status_word), _stream()), "gqla_decode_absorb_final")


def gqla_decode_absorb_paged(dims: GqlaDims, q_hat: torch.Tensor, cache: torch.Tensor, block_table: torch.Tensor,
                             page_size: int, seqlens: torch.Tensor, scale: float, num_splits: int, o_part: torch.Tensor,
                             lse_part: torch.Tensor, status_word: torch.Tensor | None = None) -> None:
    """gqla_decode_absorb over a paged cache: block_table int32 [B, max_pages] of page numbers."""
    _contig(q_hat, block_table, seqlens, o_part, lse_part)
    assert cache.dim() == 2 and cache.stride(1) == 1
    assert block_table.dtype == torch.int32 and block_table.dim() == 2 and seqlens.dtype == torch.int32
    assert o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q_hat.shape[0], q_hat.shape[1]
    _check(lib().gqla_decode_absorb_paged(ctypes.byref(dims), _dtype_code(q_hat), B, s_q, scale, num_splits, _ptr(q_hat),
                                          _ptr(cache), cache.stride(0), cache.shape[0], _ptr(block_table),
                                          block_table.shape[1], page_size, _ptr(seqlens), _ptr(o_part), _ptr(lse_part),
                                          _ptr(status_word), _stream()), "gqla_decode_absorb_paged")


def gqla_decode_gqa_paged(dims: GqlaDims, q: torch.Tensor, k_c: torch.Tensor, v: torch.Tensor, k_r: torch.Tensor,
                          block_table: torch.Tensor, page_size: int, seqlens: torch.Tensor, scale: float,
                          num_splits: int, o_part: torch.Tensor, lse_part: torch.Tensor,
                          status_word: torch.Tensor | None = None) -> None:
    """gqla_decode_gqa over paged K_C, V, k_R planes: block_table int32 [B, max_pages] of page numbers."""
    _contig(q, k_c, v, block_table, seqlens, o_part, lse_part)
    assert k_r.dim() == 2 and k_r.stride(1) == 1
    assert block_table.dtype == torch.int32 and block_table.dim() == 2 and seqlens.dtype == torch.int32
    assert o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q.shape[0], q.shape[1]
    _check(lib().gqla_decode_gqa_paged(ctypes.byref(dims), _dtype_code(q), B, s_q, scale, num_splits, _ptr(q), _ptr(k_c),
                                       _ptr(v), _ptr(k_r), k_r.stride(0), k_c.shape[0], _ptr(block_table),
                                       block_table.shape[1], page_size, _ptr(seqlens), _ptr(o_part), _ptr(lse_part),
                                       _ptr(status_word), _stream()), "gqla_decode_gqa_paged")


def gqla_append_expand(dims: GqlaDims, s_q: int, cache: torch.Tensor, seq_start: torch.Tensor, seqlens: torch.Tensor,
                       w_uk: torch.Tensor, w_uv: torch.Tensor, k_c: torch.Tensor, v: torch.Tensor,
                       k_r: torch.Tensor | None) -> None:
    """Expands only the s_q rows each sequence appended in this step (Sec. 3.1, per-token map)."""
    _contig(w_uk, w_uv, k_c, v, k_r, seq_start, seqlens)
    assert cache.dim() == 2 and cache.stride(1) == 1
    assert seq_start.dtype == torch.int64 and seqlens.dtype == torch.int32
    _check(lib().gqla_append_expand(ctypes.byref(dims), _dtype_code(cache), seqlens.shape[0], s_q, _ptr(cache),
                                    cache.stride(0), _ptr(seq_start), _ptr(seqlens), _ptr(w_uk), _ptr(w_uv), _ptr(k_c),
                                    _ptr(v), _ptr(k_r), _stream()), "gqla_append_expand")


def gqla_decode_gqa(dims: GqlaDims, q: torch.Tensor, k_c: torch.Tensor, v: torch.Tensor, k_r: torch.Tensor,
                    seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float, num_splits: int,
                    o_part: torch.Tensor, lse_part: torch.Tensor, status_word: torch.Tensor | None = None) -> None:
    """Split-KV GQA-path attention (Eq. (mha)).  k_r is [N, d_r] and may be a strided view."""
    _contig(q, k_c, v, seq_start, seqlens, o_part, lse_part)
    assert k_r.dim() == 2 and k_r.stride(1) == 1
    assert seq_start.dtype == torch.int64 and seqlens.dtype == torch.int32
    assert o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q.shape[0], q.shape[1]
    _check(lib().gqla_decode_gqa(ctypes.byref(dims), _dtype_code(q), B, s_q, scale, num_splits, _ptr(q), _ptr(k_c),
                                 _ptr(v), _ptr(k_r), k_r.stride(0), k_c.shape[0], _ptr(seq_start), _ptr(seqlens), _ptr(o_part),
                                 _ptr(lse_part), _ptr(status_word), _stream()), "gqla_decode_gqa")


def gqla_decode_gqa_noalloc(dims: GqlaDims, q: torch.Tensor, k_c: torch.Tensor, v: torch.Tensor, k_r: torch.Tensor,
                            seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float, num_splits: int,
                            out: torch.Tensor, lse: torch.Tensor | None = None,
                            status_word: torch.Tensor | None = None) -> None:
    """GQA-path step (attention + split merge) that keeps its split partials in the library's built-in
    device array instead of caller buffers, for hosts that must not allocate device memory while decoding.
    out is [B, s_q, h_q, d_h]; num_splits >= 1 (fixed plan only); raises (capacity) when
    B*num_splits*s_q*h_q > 65536 or that times d_h > 4 Mi.  Calls on one GPU share the array: keep them on
    one stream.  Call it once per device at start-up (an empty batch will do) so that the array exists
    before the host's memory manager claims the GPU."""
    _contig(q, k_c, v, seq_start, seqlens, out, lse)
    assert k_r.dim() == 2 and k_r.stride(1) == 1
    assert seq_start.dtype == torch.int64 and seqlens.dtype == torch.int32
    assert out.dtype == q.dtype and (lse is None or lse.dtype == torch.float32)
    B, s_q = q.shape[0], q.shape[1]
    _check(lib().gqla_decode_gqa_noalloc(ctypes.byref(dims), _dtype_code(q), B, s_q, scale, num_splits, _ptr(q),
                                         _ptr(k_c), _ptr(v), _ptr(k_r), k_r.stride(0), k_c.shape[0], _ptr(seq_start),
                                         _ptr(seqlens), _ptr(out), _ptr(lse), _ptr(status_word), _stream()),
           "gqla_decode_gqa_noalloc")


def gqla_combine_splits(o_part: torch.Tensor, lse_part: torch.Tensor, out: torch.Tensor,
                        lse: torch.Tensor | None = None) -> None:
    """LSE merge over the split axis: o_part [B,S,s_q,h_q,D], lse_part [B,S,s_q,h_q] -> out [B,s_q,h_q,D]."""
    _contig(o_part, lse_part, out, lse)
    B, S = o_part.shape[0], o_part.shape[1]
    rows = o_part.shape[2] * o_part.shape[3]
    _check(lib().gqla_combine_splits(B, rows, S, o_part.shape[-1], _dtype_code(out), _ptr(o_part), _ptr(lse_part),
                                     _ptr(out), _ptr(lse), _stream()), "gqla_combine_splits")


def gqla_up_proj(dims: GqlaDims, o_hat: torch.Tensor, w_uv: torch.Tensor, o: torch.Tensor) -> None:
    """o[B,s_q,h_q,d_h] = W^UV_{j(i)} o_hat  (Eq. (mqa), line 6)."""
    _contig(o_hat, w_uv, o)
    B, s_q = o_hat.shape[0], o_hat.shape[1]
    _check(lib().gqla_up_proj(ctypes.byref(dims), _dtype_code(o_hat), B, s_q, _ptr(o_hat), _ptr(w_uv), _ptr(o),
                              _stream()), "gqla_up_proj")


def gqla_combine_up_proj(dims: GqlaDims, o_part: torch.Tensor, lse_part: torch.Tensor, w_uv: torch.Tensor,
                         o: torch.Tensor, lse: torch.Tensor | None = None) -> None:
    """Split merge fused with the up-projection: o_part [B,S,s_q,h_q,r_kv], lse_part [B,S,s_q,h_q] ->
    o[B,s_q,h_q,d_h] = W^UV_{j(i)} (merged o_hat)  (Eq. (mqa), line 6)."""
    _contig(o_part, lse_part, w_uv, o, lse)
    assert o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, S, s_q = o_part.shape[0], o_part.shape[1], o_part.shape[2]
    _check(lib().gqla_combine_up_proj(ctypes.byref(dims), _dtype_code(o), B, s_q, S, _ptr(o_part), _ptr(lse_part),
                                      _ptr(w_uv), _ptr(o), _ptr(lse), _stream()), "gqla_combine_up_proj")


# ------------------------------------------------------------------ a value head dimension of its own (Sec. 3.2)


def gqla_expand_cache_dv(dims: GqlaDims, cache: torch.Tensor, w_uk: torch.Tensor, w_uv: torch.Tensor,
                         k_c: torch.Tensor, v: torch.Tensor, k_r: torch.Tensor | None) -> None:
    """gqla_expand_cache with w_uv [g, r_kv, d_v] and v [N, g, d_v]; d_v is read off w_uv."""
    _contig(w_uk, w_uv, k_c, v, k_r)
    assert cache.dim() == 2 and cache.stride(1) == 1 and v.shape[-1] == w_uv.shape[-1]
    _check(lib().gqla_expand_cache_dv(ctypes.byref(dims), w_uv.shape[-1], _dtype_code(cache), cache.shape[0], _ptr(cache),
                                      cache.stride(0), _ptr(w_uk), _ptr(w_uv), _ptr(k_c), _ptr(v), _ptr(k_r), _stream()),
           "gqla_expand_cache_dv")


def gqla_decode_gqa_dv(dims: GqlaDims, q: torch.Tensor, k_c: torch.Tensor, v: torch.Tensor, k_r: torch.Tensor,
                       seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float, num_splits: int,
                       o_part: torch.Tensor, lse_part: torch.Tensor, status_word: torch.Tensor | None = None) -> None:
    """gqla_decode_gqa with v [N, g, d_v] and o_part [B, S, s_q, h_q, d_v]; d_v is read off v."""
    _contig(q, k_c, v, seq_start, seqlens, o_part, lse_part)
    assert k_r.dim() == 2 and k_r.stride(1) == 1 and o_part.shape[-1] == v.shape[-1]
    assert seq_start.dtype == torch.int64 and seqlens.dtype == torch.int32
    assert o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q.shape[0], q.shape[1]
    _check(lib().gqla_decode_gqa_dv(ctypes.byref(dims), v.shape[-1], _dtype_code(q), B, s_q, scale, num_splits, _ptr(q),
                                    _ptr(k_c), _ptr(v), _ptr(k_r), k_r.stride(0), k_c.shape[0], _ptr(seq_start),
                                    _ptr(seqlens), _ptr(o_part), _ptr(lse_part), _ptr(status_word), _stream()),
           "gqla_decode_gqa_dv")


def gqla_up_proj_dv(dims: GqlaDims, o_hat: torch.Tensor, w_uv: torch.Tensor, o: torch.Tensor) -> None:
    """gqla_up_proj with w_uv [g, r_kv, d_v] and o [B, s_q, h_q, d_v]; d_v is read off w_uv."""
    _contig(o_hat, w_uv, o)
    assert o.shape[-1] == w_uv.shape[-1]
    B, s_q = o_hat.shape[0], o_hat.shape[1]
    _check(lib().gqla_up_proj_dv(ctypes.byref(dims), w_uv.shape[-1], _dtype_code(o_hat), B, s_q, _ptr(o_hat), _ptr(w_uv),
                                 _ptr(o), _stream()), "gqla_up_proj_dv")


# ------------------------------------------------------------------ FP8 (E4M3) cache


def gqla_quantize_cols_e4m3(src: torch.Tensor, split: int, scale_a: float, scale_b: float, dst: torch.Tensor) -> None:
    """dst (uint8 codes, dense [rows, width]) = encode(src / scale), scale_a for columns < split, scale_b beyond.
    src is [rows, width] (rows may be strided) or any dense tensor whose last dimension is the width."""
    if src.dim() != 2:
        src = src.reshape(-1, src.shape[-1])
    assert src.stride(1) == 1 and dst.dtype == torch.uint8 and dst.is_contiguous() and dst.numel() == src.numel()
    _check(lib().gqla_quantize_cols_e4m3(_dtype_code(src), src.shape[0], src.shape[1], split, scale_a, scale_b, _ptr(src),
                                         src.stride(0), _ptr(dst), _stream()), "gqla_quantize_cols_e4m3")


def gqla_quantize_rows_e4m3(src: torch.Tensor, split: int, pre_a: float, pre_b: float, dst: torch.Tensor,
                            row_scale: torch.Tensor) -> None:
    """Per-row quantisation of query rows (last dimension = width): codes into dst (uint8, same shape), the row
    scales into row_scale (fp32, shape without the last dimension)."""
    _contig(src, dst, row_scale)
    assert dst.dtype == torch.uint8 and row_scale.dtype == torch.float32
    rows = src.numel() // src.shape[-1]
    assert row_scale.numel() == rows and dst.numel() == src.numel()
    _check(lib().gqla_quantize_rows_e4m3(_dtype_code(src), rows, src.shape[-1], split, pre_a, pre_b, _ptr(src), _ptr(dst),
                                         _ptr(row_scale), _stream()), "gqla_quantize_rows_e4m3")


def gqla_decode_absorb_fp8(dims: GqlaDims, q8: torch.Tensor, q_scale: torch.Tensor, cache8: torch.Tensor, v_scale: float,
                           seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float, num_splits: int,
                           o_part: torch.Tensor, lse_part: torch.Tensor, status_word: torch.Tensor | None = None) -> None:
    """Absorb-path attention over an E4M3 latent cache (codes [N, r_kv+d_r]); q8 / q_scale from gqla_quantize_rows_e4m3."""
    _contig(q8, q_scale, seq_start, seqlens, o_part, lse_part)
    assert q8.dtype == torch.uint8 and cache8.dtype == torch.uint8 and cache8.dim() == 2 and cache8.stride(1) == 1
    assert q_scale.dtype == torch.float32 and o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q8.shape[0], q8.shape[1]
    _check(lib().gqla_decode_absorb_fp8(ctypes.byref(dims), B, s_q, scale, num_splits, _ptr(q8), _ptr(q_scale), _ptr(cache8),
                                        cache8.stride(0), cache8.shape[0], v_scale, _ptr(seq_start), _ptr(seqlens),
                                        _ptr(o_part), _ptr(lse_part), _ptr(status_word), _stream()), "gqla_decode_absorb_fp8")


def gqla_decode_absorb_fp8_final(dims: GqlaDims, q8: torch.Tensor, q_scale: torch.Tensor, cache8: torch.Tensor, v_scale: float,
                                 seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float, o_hat: torch.Tensor,
                                 lse: torch.Tensor | None = None, status_word: torch.Tensor | None = None) -> None:
    """Whole-sequence absorb-path attention over an E4M3 latent cache: bf16 o_hat [B, s_q, h_q, r_kv] for gqla_up_proj."""
    _contig(q8, q_scale, seq_start, seqlens, o_hat, lse)
    assert q8.dtype == torch.uint8 and cache8.dtype == torch.uint8 and cache8.dim() == 2 and cache8.stride(1) == 1
    assert q_scale.dtype == torch.float32 and o_hat.dtype == torch.bfloat16
    B, s_q = q8.shape[0], q8.shape[1]
    _check(lib().gqla_decode_absorb_fp8_final(ctypes.byref(dims), B, s_q, scale, _ptr(q8), _ptr(q_scale), _ptr(cache8),
                                              cache8.stride(0), cache8.shape[0], v_scale, _ptr(seq_start), _ptr(seqlens),
                                              _ptr(o_hat), _ptr(lse), _ptr(status_word), _stream()),
           "gqla_decode_absorb_fp8_final")


def gqla_decode_gqa_fp8(dims: GqlaDims, q8: torch.Tensor, q_scale: torch.Tensor, k_c8: torch.Tensor, v8: torch.Tensor,
                        k_r8: torch.Tensor, v_scale: float, seq_start: torch.Tensor, seqlens: torch.Tensor, scale: float,
                        num_splits: int, o_part: torch.Tensor, lse_part: torch.Tensor,
                        status_word: torch.Tensor | None = None) -> None:
    """GQA-path attention over E4M3 planes K_C, V [N, g, d_h] and k_R [N, d_r] (k_R rows may be strided)."""
    _contig(q8, q_scale, k_c8, v8, seq_start, seqlens, o_part, lse_part)
    assert q8.dtype == k_c8.dtype == v8.dtype == k_r8.dtype == torch.uint8 and k_r8.dim() == 2 and k_r8.stride(1) == 1
    assert q_scale.dtype == torch.float32 and o_part.dtype == torch.float32 and lse_part.dtype == torch.float32
    B, s_q = q8.shape[0], q8.shape[1]
    _check(lib().gqla_decode_gqa_fp8(ctypes.byref(dims), B, s_q, scale, num_splits, _ptr(q8), _ptr(q_scale), _ptr(k_c8),
                                     _ptr(v8), _ptr(k_r8), k_r8.stride(0), k_c8.shape[0], v_scale, _ptr(seq_start),
                                     _ptr(seqlens), _ptr(o_part), _ptr(lse_part), _ptr(status_word), _stream()),
           "gqla_decode_gqa_fp8")


# ------------------------------------------------------------------ integer helpers (host)


def gqla_split_plan(seqlen: int, num_splits: int) -> list[tuple[int, int]]:
    begin = (c_int32 * num_splits)()
    end = (c_int32 * num_splits)()
    _check(lib().gqla_split_plan(seqlen, num_splits, begin, end), "gqla_split_plan")
    return [(int(begin[k]), int(end[k])) for k in range(num_splits)]


def gqla_balanced_plan(seqlens, s_cap: int, workers: int):
    """Balanced split plan of a batch: (plans, owners) with plans[b] = s_cap (begin, end) row ranges
    ((0, 0) = unused slot) and owners[b][k] the worker that produces the slot (-1 = unused)."""
    n = len(seqlens)
    sl = (c_int32 * max(n, 1))(*[int(t) for t in seqlens])
    begin = (c_int32 * max(n * s_cap, 1))()
    end = (c_int32 * max(n * s_cap, 1))()
    own = (c_int32 * max(n * s_cap, 1))()
    _check(lib().gqla_balanced_plan(sl, n, s_cap, workers, begin, end, own), "gqla_balanced_plan")
    plans = [[(int(begin[b * s_cap + k]), int(end[b * s_cap + k])) for k in range(s_cap)] for b in range(n)]
    owners = [[int(own[b * s_cap + k]) for k in range(s_cap)] for b in range(n)]
    return plans, owners


def gqla_balanced_workers(dims: GqlaDims, dtype: torch.dtype, s_q: int, path: str) -> int:
    """Workers a balanced decode call is cut for on the current device (0: fixed plan is used instead)."""
    code = GQLA_BF16 if dtype == torch.bfloat16 else GQLA_F32
    return int(lib().gqla_balanced_workers(ctypes.byref(dims), code, s_q, 0 if path == "absorb" else 1))


def gqla_visible_limit(seqlen: int, s_q: int, p: int) -> int:
    return int(lib().gqla_visible_limit(seqlen, s_q, p))


def gqla_group_of_head(dims: GqlaDims, head: int) -> int:
    return int(lib().gqla_group_of_head(ctypes.byref(dims), head))
