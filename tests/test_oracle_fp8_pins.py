"""Pins for the oracle's FP8 (E4M3) functions: the code table against the format's published bit patterns and a
library conversion, the rounding against hand-worked ties, saturation, a brute-force nearest search, and the
quantised decode paths against the existing (pinned) oracle on explicitly decoded inputs."""
import numpy as np
import pytest
import torch

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import synth


def test_code_table_matches_published_bit_patterns_and_library():
    # hand values: 0, smallest subnormal 2^-9, smallest normal 2^-6, 1.0, 1.5, 2.0, largest finite 448, negative zero, -1.0
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x3C: 1.5, 0x40: 2.0, 0x7E: 448.0,
            0xB8: -1.0, 0xFE: -448.0, 0x77: 240.0}
    for c, v in hand.items():
        assert O.e4m3_decode(np.array([c], dtype=np.uint8))[0] == v, hex(c)
    assert np.isnan(O.e4m3_decode(np.array([0x7F, 0xFF], dtype=np.uint8))).all()
    allc = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(allc).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = O.e4m3_decode(allc)
    assert np.array_equal(np.isnan(got), np.isnan(lib))
    assert np.array_equal(got[~np.isnan(got)], lib[~np.isnan(lib)])
    # strictly increasing over the non-negative finite codes, 127 of them
    pos = got[:127]
    assert (np.diff(pos) > 0).all() and pos[0] == 0 and pos[-1] == 448


def test_encode_round_trip_ties_and_saturation():
    allc = np.arange(256, dtype=np.uint8)
    finite = allc[~np.isnan(O.e4m3_decode(allc))]
    back = O.e4m3_encode(O.e4m3_decode(finite).astype(np.float32))
    keep = finite != 0x80  # -0.0 encodes with its sign kept
    assert np.array_equal(back[keep], finite[keep]) and back[~keep][0] in (0x00, 0x80)
    # hand-worked ties: 1.0625 is halfway 1.0 (0x38, even) / 1.125 (0x39); 1.1875 halfway 1.125 (0x39) / 1.25 (0x3A, even)
    # 2^-10 halfway 0 / 2^-9 -> 0;  3 * 2^-10 halfway 2^-9 (0x01) / 2^-8 (0x02, even)
    x = np.array([1.0625, 1.1875, 2.0 ** -10, 3 * 2.0 ** -10, -1.0625, 1.0626, 1.0624], dtype=np.float32)
    assert list(O.e4m3_encode(x)) == [0x38, 0x3A, 0x00, 0x02, 0xB8, 0x39, 0x38]
    # saturation: no infinity in the format, everything beyond 448 gives 448; 464 is the tie towards the missing 480
    big = np.array([448.0, 449.0, 464.0, 465.0, 1e6, -1e30, np.inf], dtype=np.float32)
    assert list(O.e4m3_encode(big)) == [0x7E, 0x7E, 0x7E, 0x7E, 0x7E, 0xFE, 0x7E]
    assert O.e4m3_encode(np.array([np.nan], dtype=np.float32))[0] == 0x7F


def test_encode_against_library_and_brute_force_nearest():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(20000) * 3, rng.standard_normal(5000) * 100, rng.standard_normal(5000) * 1e-2,
                        rng.uniform(-448, 448, 5000)]).astype(np.float32)
    x = x[np.abs(x) <= 448]
    got = O.e4m3_encode(x)
    lib = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    zero = (got & 0x7F) == 0
    assert np.array_equal(got[~zero], lib[~zero]) and np.array_equal(got[zero] & 0x7F, lib[zero] & 0x7F)
    # brute force on a sample: no representable value is closer
    grid = O.e4m3_decode(np.arange(127, dtype=np.uint8))
    for v, c in zip(x[:300].astype(np.float64), got[:300]):
        err = abs(abs(v) - grid[c & 0x7F])
        assert err <= np.abs(abs(v) - grid).min() + 0.0
    # relative error bound in the normal range: half a unit in the 4th significant bit
    dec = O.e4m3_decode(got)
    normal = np.abs(x) >= 2.0 ** -6
    assert (np.abs(dec[normal] - x[normal]) <= 2.0 ** -4 * np.abs(x[normal])).all()


def test_column_and_row_quantisers():
    rng = np.random.default_rng(5)
    x = torch.from_numpy(rng.standard_normal((7, 12)).astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    codes = O.quantize_cols_e4m3(x, 8, 0.25, 0.5)
    # columns < 8 were divided by 0.25, the others by 0.5 (exact in fp32 for these powers of two)
    ref = torch.from_numpy(np.concatenate([x[:, :8] * 4, x[:, 8:] * 2], 1)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(codes & 0x7F, ref & 0x7F)
    # values already on the scaled grid survive the round trip exactly
    g = O.e4m3_decode(rng.integers(0, 127, size=(5, 6)).astype(np.uint8)) * 0.125
    assert np.array_equal(O.e4m3_decode(O.quantize_cols_e4m3(g, 6, 0.125, 1.0)) * 0.125, g)
    # rows: the largest magnitude of every row lands on +-448, an all-zero row gets scale 1 and codes 0
    x[3] = 0
    c8, s = O.quantize_rows_e4m3(x, 8, 2.0, 0.5)
    y = np.concatenate([x[:, :8] * 2.0, x[:, 8:] * 0.5], 1)
    assert s.dtype == np.float32 and s[3] == 1.0 and (c8[3] & 0x7F == 0).all()
    live = np.arange(7) != 3
    assert (np.abs(O.e4m3_decode(c8)).max(axis=1)[live] == 448).all()
    np.testing.assert_allclose(s[live], np.abs(y).max(axis=1)[live] / 448, rtol=1e-6)
    deq = O.e4m3_decode(c8) * s[:, None]
    assert (np.abs(deq - y) <= 2.0 ** -4 * np.abs(y) + 2.0 ** -10 * s[:, None] * 448 / 448).all()


@pytest.mark.parametrize("s_q,S", [(1, 1), (2, 3)])
def test_fp8_decode_paths_equal_the_plain_oracle_on_decoded_inputs(s_q, S):
    """The FP8 decode functions are the pinned bf16/fp64 functions applied to explicitly decoded numbers: feed the
    plain functions hand-decoded inputs (a torch library conversion, not the oracle's own table) and compare."""
    w = synth.Workload("f8", 8, 2, 16, 32, 8, batch=2, s_q=s_q, dtype="bf16", seed=21)
    x = synth.make_inputs(w, seqlens=np.array([70, 129], dtype=np.int32), q_gain=2.0)
    d = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    f = {k: synth.to_f64(t) for k, t in x.items() if k not in ("seq_start", "seqlens")}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    sc, sr = 0.02, 0.01
    cache8 = O.quantize_cols_e4m3(f["cache"], w.r_kv, sc, sr)
    qh = O.absorb_q(d, f["q_c"], f["q_r"], f["w_uk"])
    q8, qs = O.quantize_rows_e4m3(qh, w.r_kv, sc, sr)
    o, l = O.decode_absorb_fp8_partials(d, q8, qs, cache8, sc, ss, sl, s_q, w.scale, S)
    lib_dec = lambda c: torch.from_numpy(np.ascontiguousarray(c)).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    o2, l2 = O.decode_absorb_partials(d, lib_dec(q8) * qs.astype(np.float64)[..., None], lib_dec(cache8), ss, sl, s_q, w.scale, S)
    np.testing.assert_allclose(o, o2 * sc, rtol=1e-13, atol=0)
    np.testing.assert_array_equal(l, l2)
    # and it approximates the unquantised attention: scores differ by the two roundings (relative 2^-4 each)
    o_ref, _ = O.decode_absorb_partials(d, qh, f["cache"], ss, sl, s_q, w.scale, S)
    assert np.abs(o - o_ref).max() <= 0.25 * np.abs(o_ref).max()
    # GQA planes
    kc, v, kr = O.expand_cache(d, f["cache"], f["w_uk"], f["w_uv"])
    sk, sv = 0.03, 0.04
    kc8 = O.quantize_cols_e4m3(kc, w.d_h, sk, sk)
    v8 = O.quantize_cols_e4m3(v, w.d_h, sv, sv)
    kr8 = O.quantize_cols_e4m3(kr, w.d_r, sr, sr)
    q = np.concatenate([f["q_c"], f["q_r"]], -1)
    q8g, qsg = O.quantize_rows_e4m3(q, w.d_h, sk, sr)
    og, lg = O.decode_gqa_fp8_partials(d, q8g, qsg, kc8, v8, kr8, sv, ss, sl, s_q, w.scale, S)
    og2, lg2 = O.decode_gqa_partials(d, lib_dec(q8g) * qsg.astype(np.float64)[..., None], lib_dec(kc8), lib_dec(v8), lib_dec(kr8),
                                     ss, sl, s_q, w.scale, S)
    np.testing.assert_allclose(og, og2 * sv, rtol=1e-13, atol=0)
    np.testing.assert_array_equal(lg, lg2)
    og_ref, _ = O.decode_gqa_partials(d, q, kc, v, kr, ss, sl, s_q, w.scale, S)
    assert np.abs(og - og_ref).max() <= 0.25 * np.abs(og_ref).max()
