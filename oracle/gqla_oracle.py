"""fp64 CPU oracle for the GQLA decode hot path.  TEST INFRASTRUCTURE ONLY.

This module is the checker, not the product: only the test-suite, the smoke
check and the benchmark's CPU-baseline leg may import it.  It shares no code
with the CUDA library (no common headers, helpers, tables or constants) and it
never imports the package that wraps that library.

Everything is the plain definition of the operation, written out in numpy
float64 with no blocking, fusion or reordering beyond what the paper's
equations state.  A numpy matmul serves as the contraction step.

Notation (paper Sec. 3.1 "Group-Query Latent Attention"):
    h_q   query heads                g     K/V groups
    d_h   per-head dim               r_kv  latent rank
    d_r   decoupled-RoPE dim (d_h^R) hpg   h_q / g heads per group
    c     latent c^KV  [.., r_kv]    k_r   shared RoPE key k^R [.., d_r]
    W_UK, W_UV  stored as [g, r_kv, d_h]; W[j, r, d] is entry (d, r) of the
                paper's group-j slice  W_j in R^{d_h x r_kv}.
    d_v   value head dim d_h^V.  Sec. 3.1 gives W^UV the shape of W^UK (d_v = d_h); the
          MLA -> GQLA factorisation of Sec. 3.2 carries a separate one
          (W~^UKV in R^{g (d_h + d_h^V) x r_kv}).  It is read off the arrays: W_UV is
          [g, r_kv, d_v], V is [N, g, d_v], outputs are d_v wide; Dims.d_v (0 = d_h)
          only enters the cache-size accounting.

Every function is pinned by tests/test_oracle_pins.py (the FP8 ones by tests/test_oracle_fp8_pins.py) to something other than
itself (brute force over python loops, closed forms, invariants, the two-path
equivalence the paper states, the printed Roofline table).  Nothing here is
"parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

NEG_INF = -np.inf

# --------------------------------------------------------------------------
# integer bookkeeping
# --------------------------------------------------------------------------


@dataclass(frozen=True)
class Dims:
    """The (h_q, g, d_h, r_kv, d_h^R) tuple of Sec. 4.2 (canonical: 128, 8, 128, 512, 64)."""

    h_q: int
    g: int
    d_h: int
    r_kv: int
    d_r: int
    d_v: int = 0  # value head dim d_h^V of Sec. 3.2; 0 means d_h (Sec. 3.1)

    @property
    def dv(self) -> int:
        return self.d_v if self.d_v > 0 else self.d_h

    @property
    def hpg(self) -> int:
        assert self.h_q % self.g == 0
        return self.h_q // self.g


def group_of_head(dims: Dims, i: int) -> int:
    """Head -> group routing, Sec. 3.1 "GQA path": j(i) = ceil(i / (h_q/g)) with
    1-indexed i and j.  Argument and result here are 0-indexed."""
    i1 = i + 1
    j1 = -(-i1 // dims.hpg)  # ceil
    return j1 - 1


def visible_limit(seqlen: int, s_q: int, p: int) -> int:
    """Number of cache rows query p (0..s_q-1) of a step may attend.

    Eq. (mha)/(mqa) sum over s = 1..t: the query at position t sees positions
    <= t, itself included.  The s_q new tokens are already appended, seqlen
    counts them, and query p sits at (0-indexed) position seqlen - s_q + p, so
    it sees rows [0, seqlen - (s_q - 1 - p)).  Clipped at zero.
    """
    return max(0, seqlen - (s_q - 1 - p))


SPLIT_GRANULE = 64


def split_plan(seqlen: int, num_splits: int) -> list[tuple[int, int]]:
    """Split-KV partition (not in the paper; a reading fixed by this build).

    chunk = ceil(ceil(seqlen / S) / 64) * 64 tokens; split k covers
    [k*chunk, min((k+1)*chunk, seqlen)), possibly empty (begin == end).
    """
    assert num_splits >= 1 and seqlen >= 0
    per = -(-seqlen // num_splits)
    chunk = -(-per // SPLIT_GRANULE) * SPLIT_GRANULE
    out = []
    for k in range(num_splits):
        b = min(k * chunk, seqlen)
        e = min((k + 1) * chunk, seqlen)
        out.append((b, e))
    return out


TILE_ROWS = 128


def balanced_plan(seqlens, num_splits: int, workers: int) -> list[list[tuple[int, int]]]:
    """Balanced split-KV partition of a whole batch (not in the paper; a reading fixed by this build).

    The 128-row tiles of all sequences are numbered end to end, sequence 0 first.  Tile number n goes to
    worker n // share with share = max(ceil(total / workers), ceil(max_b tiles_b / (S - 1)), 1).  The tiles
    of one sequence that one worker holds form one piece; a sequence's pieces are numbered in row order
    and its unused slots are empty, written (0, 0).  Returned: per sequence, S (begin, end) row ranges.
    Stated tile by tile on purpose: no closed forms shared with the library's arithmetic."""
    S = num_splits
    assert S >= 2 and workers >= 1
    tiles = [(-(-int(T) // TILE_ROWS) if T > 0 else 0) for T in seqlens]
    total = sum(tiles)
    share = max(-(-total // workers), -(-max(tiles + [0]) // (S - 1)), 1)
    plans = []
    n = 0
    for T, nt in zip(seqlens, tiles):
        by_worker = {}
        for i in range(nt):
            by_worker.setdefault((n + i) // share, []).append(i)
        n += nt
        pieces = []
        for wkr in sorted(by_worker):
            idx = by_worker[wkr]
            assert idx == list(range(idx[0], idx[-1] + 1))
            pieces.append((idx[0] * TILE_ROWS, min((idx[-1] + 1) * TILE_ROWS, int(T))))
        assert len(pieces) <= S
        plans.append(pieces + [(0, 0)] * (S - len(pieces)))
    return plans


# --------------------------------------------------------------------------
# the three plain contractions (absorb q, expand cache, up-project)
# --------------------------------------------------------------------------


def absorb_q(dims: Dims, q_c: np.ndarray, q_r: np.ndarray, w_uk: np.ndarray) -> np.ndarray:
    """Eq. (mqa), second line: q_hat_i = [ (W^UK_{j(i)})^T q^C_i ; q^R_i ].

    q_c [B, s_q, h_q, d_h], q_r [B, s_q, h_q, d_r], w_uk [g, r_kv, d_h]
    -> q_hat [B, s_q, h_q, r_kv + d_r].
    """
    B, s_q, h_q, _ = q_c.shape
    out = np.zeros((B, s_q, h_q, dims.r_kv + dims.d_r), dtype=np.float64)
    for i in range(h_q):
        j = group_of_head(dims, i)
        # (W_j)^T q : contract over d, W stored [r, d]
        out[:, :, i, : dims.r_kv] = q_c[:, :, i, :].astype(np.float64) @ w_uk[j].astype(np.float64).T
        out[:, :, i, dims.r_kv:] = q_r[:, :, i, :]
    return out


def expand_cache(dims: Dims, cache: np.ndarray, w_uk: np.ndarray, w_uv: np.ndarray):
    """Sec. 3.1: k^C = W^UK c^KV, v^C = W^UV c^KV per group; k^R carried over.

    cache [N, r_kv + d_r] -> K_C [N, g, d_h], V [N, g, d_v], k_R [N, d_r]  (w_uv is [g, r_kv, d_v]).
    """
    c = cache[:, : dims.r_kv].astype(np.float64)
    N = c.shape[0]
    k_c = np.zeros((N, dims.g, dims.d_h), dtype=np.float64)
    v = np.zeros((N, dims.g, w_uv.shape[2]), dtype=np.float64)
    for j in range(dims.g):
        k_c[:, j, :] = c @ w_uk[j].astype(np.float64)  # sum_r W[j,r,d] c[r]
        v[:, j, :] = c @ w_uv[j].astype(np.float64)
    k_r = cache[:, dims.r_kv:].astype(np.float64).copy()
    return k_c, v, k_r


def up_proj(dims: Dims, o_hat: np.ndarray, w_uv: np.ndarray) -> np.ndarray:
    """Eq. (mqa): o_i = W^UV_{j(i)} o_hat_i.  o_hat [B, s_q, h_q, r_kv] -> [B, s_q, h_q, d_v]."""
    B, s_q, h_q, _ = o_hat.shape
    out = np.zeros((B, s_q, h_q, w_uv.shape[2]), dtype=np.float64)
    for i in range(h_q):
        j = group_of_head(dims, i)
        out[:, :, i, :] = o_hat[:, :, i, :].astype(np.float64) @ w_uv[j].astype(np.float64)
    return out


# --------------------------------------------------------------------------
# softmax attention over a key range: the definition
# --------------------------------------------------------------------------


def _attend(q: np.ndarray, K: np.ndarray, V: np.ndarray, scale: float, lo: int, hi: int):
    """softmax_s(scale * q.k_s) over rows s in [lo, hi) of K, applied to V.

    q [R, D], K [T, D], V [T, Dv].  Returns (o [R, Dv], lse [R]) with lse the
    natural-log-sum-exp of the scaled scores.  An empty range gives o = 0 and
    lse = -inf (there is nothing to normalise)."""
    R = q.shape[0]
    if hi <= lo:
        return np.zeros((R, V.shape[1])), np.full((R,), NEG_INF)
    x = scale * (q @ K[lo:hi].T)  # [R, n]
    m = x.max(axis=1, keepdims=True)
    e = np.exp(x - m)
    l = e.sum(axis=1, keepdims=True)
    o = (e / l) @ V[lo:hi]
    lse = (m + np.log(l))[:, 0]
    return o, lse


def _decode(dims, q_rows_of, K_of, V_of, Dv, B, s_q, seq_start, seqlens, scale, num_splits, plans=None):
    """Shared driver for the two paths: loops (b, split, p) and calls the
    definition on the rows each query may see.  q_rows_of(b, p) -> list of
    (head slice, q [n, D]); K_of/V_of (b, head slice) -> arrays over the
    sequence's rows."""
    h_q = dims.h_q
    S = num_splits
    o_part = np.zeros((B, S, s_q, h_q, Dv), dtype=np.float64)
    lse_part = np.full((B, S, s_q, h_q), NEG_INF, dtype=np.float64)
    for b in range(B):
        T = int(seqlens[b])
        plan = split_plan(T, S) if plans is None else plans[b]
        assert len(plan) == S
        for p in range(s_q):
            lim = visible_limit(T, s_q, p)
            for hs, q in q_rows_of(b, p):
                K = K_of(b, hs)
                V = V_of(b, hs)
                for k, (sb, se) in enumerate(plan):
                    o, lse = _attend(q, K, V, scale, sb, min(se, lim))
                    o_part[b, k, p, hs, :] = o
                    lse_part[b, k, p, hs] = lse
    return o_part, lse_part


def decode_absorb_partials(dims: Dims, q_hat, cache, seq_start, seqlens, s_q, scale, num_splits, plans=None):
    """Eq. (mqa): k_hat_s = [c_s ; k^R_s], v_hat_s = c_s, all heads share them.

    q_hat [B, s_q, h_q, r_kv+d_r]; cache [N, r_kv+d_r]; sequence b owns rows
    seq_start[b] .. seq_start[b]+seqlens[b]-1.  Returns per-split partials
    o_part [B, S, s_q, h_q, r_kv] (each normalised within its split) and
    lse_part [B, S, s_q, h_q]."""
    B = q_hat.shape[0]
    r = dims.r_kv
    q64 = q_hat.astype(np.float64)

    def rows(b):
        s0 = int(seq_start[b])
        return cache[s0: s0 + int(seqlens[b])].astype(np.float64)

    memo = {}

    def K_of(b, hs):
        if memo.get("b") != b:
            memo["b"], memo["K"] = b, rows(b)
        return memo["K"]

    def V_of(b, hs):
        return K_of(b, hs)[:, :r]

    def q_rows_of(b, p):
        return [(slice(0, dims.h_q), q64[b, p])]

    return _decode(dims, q_rows_of, K_of, V_of, r, B, s_q, seq_start, seqlens, scale, num_splits, plans)


def decode_gqa_partials(dims: Dims, q, k_c, v, k_r, seq_start, seqlens, s_q, scale, num_splits, plans=None):
    """Eq. (mha): head i attends k_{s,i} = [k^C_{s,j(i)} ; k^R_s] with values v^C_{s,j(i)}.

    q [B, s_q, h_q, d_h+d_r]; k_c [N, g, d_h]; v [N, g, d_v]; k_r [N, d_r]."""
    B = q.shape[0]
    q64 = q.astype(np.float64)
    hpg = dims.hpg

    def span(b):
        s0 = int(seq_start[b])
        return slice(s0, s0 + int(seqlens[b]))

    def group(hs):
        j = group_of_head(dims, hs.start)
        assert group_of_head(dims, hs.stop - 1) == j
        return j

    def K_of(b, hs):
        sp = span(b)
        return np.concatenate([k_c[sp, group(hs), :].astype(np.float64), k_r[sp].astype(np.float64)], axis=1)

    def V_of(b, hs):
        return v[span(b), group(hs), :].astype(np.float64)

    def q_rows_of(b, p):
        return [(slice(j * hpg, (j + 1) * hpg), q64[b, p, j * hpg:(j + 1) * hpg]) for j in range(dims.g)]

    return _decode(dims, q_rows_of, K_of, V_of, v.shape[2], B, s_q, seq_start, seqlens, scale, num_splits, plans)


def unpage(paged: np.ndarray, block_table: np.ndarray, page_size: int, seqlens: np.ndarray):
    """Paged cache -> packed cache (paging is storage only; the paper's model leaves it out, Sec. 5.1).

    Row t of sequence b lives in row block_table[b, t // page_size] * page_size + t % page_size of
    `paged` [n_pages * page_size, ...].  Returns (packed rows of all sequences in order, seq_start), so
    that every function above applies unchanged."""
    rows, seq_start, n = [], np.zeros(len(seqlens), dtype=np.int64), 0
    for b, T in enumerate(seqlens):
        seq_start[b] = n
        for t in range(int(T)):
            rows.append(int(block_table[b, t // page_size]) * page_size + t % page_size)
        n += int(T)
    return paged[np.array(rows, dtype=np.int64)], seq_start


def combine_splits(o_part: np.ndarray, lse_part: np.ndarray):
    """Log-sum-exp merge of per-split partials (split axis = 1).

    M = max_k lse_k, w_k = exp(lse_k - M), o = sum_k w_k o_k / sum_k w_k,
    lse = M + ln sum_k w_k.  Rows whose every split is empty give o = 0,
    lse = -inf.  o_part [B, S, ..., D], lse_part [B, S, ...]."""
    M = lse_part.max(axis=1, keepdims=True)
    dead = ~np.isfinite(M)
    Msafe = np.where(dead, 0.0, M)
    w = np.exp(lse_part - Msafe)  # exp(-inf) = 0 for empty splits
    den = w.sum(axis=1, keepdims=True)
    den_safe = np.where(den == 0.0, 1.0, den)
    o = (w[..., None] * o_part).sum(axis=1) / den_safe[:, 0][..., None]
    with np.errstate(divide="ignore"):
        lse = (Msafe + np.log(den))[:, 0]
    lse = np.where(dead[:, 0], NEG_INF, lse)
    return o, lse


def decode_absorb(dims, q_hat, cache, seq_start, seqlens, s_q, scale):
    """Whole-sequence absorb-path attention: o_hat [B, s_q, h_q, r_kv], lse."""
    o, l = decode_absorb_partials(dims, q_hat, cache, seq_start, seqlens, s_q, scale, 1)
    return o[:, 0], l[:, 0]


def decode_gqa(dims, q, k_c, v, k_r, seq_start, seqlens, s_q, scale):
    """Whole-sequence GQA-path attention: o [B, s_q, h_q, d_h], lse."""
    o, l = decode_gqa_partials(dims, q, k_c, v, k_r, seq_start, seqlens, s_q, scale, 1)
    return o[:, 0], l[:, 0]


# --------------------------------------------------------------------------
# FP8 (E4M3) cache: the paper leaves KV-cache quantisation out of its model (Limitations, item (i)); the
# format, the scales and the rounding are this library's reading (element type: the 8-bit float with 4
# exponent bits (bias 7), 3 mantissa bits, no infinities, largest finite value 448, NaN = S.1111.111).
# --------------------------------------------------------------------------

E4M3_MAX = 448.0


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """Value of every 8-bit code, written out from the format's definition:
    sign s, exponent field e (4 bits), mantissa field m (3 bits);
    e = 0: (-1)^s 2^-6 (m/8)   (subnormal);   e > 0: (-1)^s 2^(e-7) (1 + m/8);   e = 15, m = 7: NaN."""
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where((c >> 7) & 1, -1.0, 1.0)
    e = (c >> 3) & 15
    m = c & 7
    val = np.where(e == 0, 2.0 ** -6 * (m / 8.0), 2.0 ** (e - 7.0) * (1.0 + m / 8.0))
    val = np.where((e == 15) & (m == 7), np.nan, val)
    return sign * val


def e4m3_encode(y: np.ndarray) -> np.ndarray:
    """fp32 -> code: round to the nearest representable value, ties to the code with an even mantissa
    field, magnitudes beyond 448 saturate to 448 (no infinity exists), NaN -> 0x7F.
    Brute statement: among the 127 non-negative finite values pick the closest one to |y|."""
    y = np.asarray(y, dtype=np.float32).astype(np.float64)  # fp32 values are exact in fp64
    grid = e4m3_decode(np.arange(127, dtype=np.uint8))  # codes 0..126: 0 .. 448, increasing
    a = np.minimum(np.abs(y), E4M3_MAX)
    hi = np.clip(np.searchsorted(grid, a, side="left"), 0, 126)  # first grid value >= a
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - grid[lo], grid[hi] - a
    pick_lo = (d_lo < d_hi) | ((d_lo == d_hi) & (lo % 2 == 0))
    code = np.where(pick_lo, lo, hi).astype(np.int64)
    code = np.where(np.signbit(y), code | 0x80, code)
    code = np.where(np.isnan(y), 0x7F, code)
    return code.astype(np.uint8)


def quantize_cols_e4m3(x: np.ndarray, split: int, scale_a: float, scale_b: float) -> np.ndarray:
    """Per-tensor-plane quantisation of a stored tensor [..., width]: columns < split carry scale_a, the
    others scale_b;  code = encode( fp32(x) * fp32(1 / scale) ), every step rounded to fp32 (the decision
    that picks an integer code is taken in fp32 on both sides of a comparison)."""
    x32 = np.asarray(x, dtype=np.float32)
    inv = np.empty(x32.shape[-1], dtype=np.float32)
    inv[:split] = np.float32(1.0) / np.float32(scale_a)
    inv[split:] = np.float32(1.0) / np.float32(scale_b)
    return e4m3_encode(x32 * inv)


def quantize_rows_e4m3(x: np.ndarray, split: int, pre_a: float, pre_b: float):
    """Per-row quantisation of query rows [..., width]: y = fp32(x) * pre (pre_a on columns < split, pre_b
    on the others: the cache planes' scales, folded into the query so that scores need no per-column
    factor), s = max|y| / 448 (1 for an all-zero row), code = encode(y * fp32(1 / s)).  Returns (codes,
    s as fp32 [...]).  All arithmetic in fp32."""
    x32 = np.asarray(x, dtype=np.float32)
    pre = np.empty(x32.shape[-1], dtype=np.float32)
    pre[:split] = np.float32(pre_a)
    pre[split:] = np.float32(pre_b)
    y = x32 * pre
    amax = np.abs(y).max(axis=-1)
    s = np.where(amax > 0, amax / np.float32(E4M3_MAX), np.float32(1.0)).astype(np.float32)
    inv = (np.float32(1.0) / s).astype(np.float32)
    return e4m3_encode(y * inv[..., None]), s


def decode_absorb_fp8_partials(dims: Dims, q8, q_scale, cache8, v_scale, seq_start, seqlens, s_q, scale, num_splits,
                               plans=None):
    """Eq. (mqa), lines 3-5, on an E4M3 latent cache.  Scores  x_s = scale * q_scale[row] * sum_c dec(q8)[c] dec(k8_s)[c],
    values  v_s = v_scale * dec(cache8_s)[: r_kv].  The plain definition on the decoded numbers (fp64)."""
    q = e4m3_decode(q8) * np.asarray(q_scale, dtype=np.float64)[..., None]
    o, l = decode_absorb_partials(dims, q, e4m3_decode(cache8), seq_start, seqlens, s_q, scale, num_splits, plans)
    return o * float(v_scale), l


def decode_gqa_fp8_partials(dims: Dims, q8, q_scale, k_c8, v8, k_r8, v_scale, seq_start, seqlens, s_q, scale,
                            num_splits, plans=None):
    """Eq. (mha) on E4M3 planes K_C, V, k_R; same conventions as decode_absorb_fp8_partials."""
    q = e4m3_decode(q8) * np.asarray(q_scale, dtype=np.float64)[..., None]
    o, l = decode_gqa_partials(dims, q, e4m3_decode(k_c8), e4m3_decode(v8), e4m3_decode(k_r8), seq_start, seqlens, s_q,
                               scale, num_splits, plans)
    return o * float(v_scale), l


# --------------------------------------------------------------------------
# the two end-to-end paths (same weights, same latent)
# --------------------------------------------------------------------------


def absorb_path(dims, q_c, q_r, w_uk, w_uv, cache, seq_start, seqlens, s_q, scale):
    """Eq. (mqa) up to (not including) W^O: o [B, s_q, h_q, d_h]."""
    qh = absorb_q(dims, q_c, q_r, w_uk)
    oh, _ = decode_absorb(dims, qh, cache, seq_start, seqlens, s_q, scale)
    return up_proj(dims, oh, w_uv)


def gqa_path(dims, q_c, q_r, w_uk, w_uv, cache, seq_start, seqlens, s_q, scale):
    """Eq. (mha) up to (not including) W^O: o [B, s_q, h_q, d_h]."""
    k_c, v, k_r = expand_cache(dims, cache, w_uk, w_uv)
    q = np.concatenate([q_c.astype(np.float64), q_r.astype(np.float64)], axis=-1)
    o, _ = decode_gqa(dims, q, k_c, v, k_r, seq_start, seqlens, s_q, scale)
    return o


def brute_force_path(dims, q_c, q_r, w_uk, w_uv, cache, seq_start, seqlens, s_q, scale):
    """Third, structurally different evaluation for tiny inputs: python loops.

    Materialises per-HEAD keys and values with the replicated weights of
    Eq. (mqa) line 1 (W_hat = repeat(W, h_q/g)), builds every score one dot
    product at a time, and does a two-pass softmax with math.exp."""
    B = q_c.shape[0]
    h_q, g, d_h, r, d_r = dims.h_q, dims.g, dims.d_h, dims.r_kv, dims.d_r
    d_v = w_uv.shape[2]
    reps = h_q // g
    # repeat(W, h_q/g): head i uses slice i of the group-wise replicated stack
    w_uk_hat = [w_uk[jj] for jj in range(g) for _ in range(reps)]
    w_uv_hat = [w_uv[jj] for jj in range(g) for _ in range(reps)]
    out = np.zeros((B, s_q, h_q, d_v))
    for b in range(B):
        T = int(seqlens[b])
        s0 = int(seq_start[b])
        for p in range(s_q):
            t = T - s_q + p  # 0-indexed position of this query
            for i in range(h_q):
                Wk, Wv = w_uk_hat[i], w_uv_hat[i]
                xs, vs = [], []
                for s in range(0, t + 1):  # sum_{s=1}^{t}, 1-indexed, inclusive
                    if s < 0 or s >= T:
                        continue
                    row = cache[s0 + s]
                    kc = [sum(float(Wk[rr, d]) * float(row[rr]) for rr in range(r)) for d in range(d_h)]
                    vc = [sum(float(Wv[rr, d]) * float(row[rr]) for rr in range(r)) for d in range(d_v)]
                    dot = sum(float(q_c[b, p, i, d]) * kc[d] for d in range(d_h))
                    dot += sum(float(q_r[b, p, i, d]) * float(row[r + d]) for d in range(d_r))
                    xs.append(scale * dot)
                    vs.append(vc)
                if not xs:
                    continue
                m = max(xs)
                es = [math.exp(x - m) for x in xs]
                Z = sum(es)
                for d in range(d_v):
                    out[b, p, i, d] = sum(es[n] * vs[n][d] for n in range(len(xs))) / Z
    return out


# --------------------------------------------------------------------------
# analytic accounting of Sec. 4.2 (Eqs. mqa-bytes-tok .. gqa-ai, Table "roofline")
# --------------------------------------------------------------------------


def mqa_cache_elems(dims: Dims) -> int:
    """N^tok_MQA = r_kv + d_h^R."""
    return dims.r_kv + dims.d_r


def gqa_cache_elems(dims: Dims) -> int:
    """N^tok_GQA = 2 g d_h + d_h^R; with a separate value dim (Sec. 3.2) g (d_h + d_h^V) + d_h^R."""
    return dims.g * (dims.d_h + dims.dv) + dims.d_r


def mqa_bytes(dims: Dims, L: int, bytes_per_elem: int = 2) -> int:
    """B_MQA = 2 L (r_kv + d_h^R) in BF16; independent of s_q."""
    return bytes_per_elem * L * mqa_cache_elems(dims)


def gqa_bytes(dims: Dims, L: int, bytes_per_elem: int = 2) -> int:
    """B_GQA = 2 L (2 g d_h + d_h^R) in BF16."""
    return bytes_per_elem * L * gqa_cache_elems(dims)


def mqa_flops(dims: Dims, L: int, s_q: int) -> int:
    """F_MQA = 2 L h_q s_q (2 r_kv + d_h^R)."""
    return 2 * L * dims.h_q * s_q * (2 * dims.r_kv + dims.d_r)


def gqa_flops(dims: Dims, L: int, s_q: int) -> int:
    """F_GQA = 2 L h_q s_q (2 d_h + d_h^R); with a separate value dim d_h + d_h^V + d_h^R per (head, key)."""
    return 2 * L * dims.h_q * s_q * (dims.d_h + dims.dv + dims.d_r)


def roofline_step(flops: float, nbytes: float, peak_flops: float, bw: float):
    """Table "roofline" caption: time = max(F / FLOPs_max, B / BW).  Returns (mem_s, cmp_s, step_s)."""
    mem = nbytes / bw
    cmp_ = flops / peak_flops
    return mem, cmp_, max(mem, cmp_)
