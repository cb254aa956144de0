"""Pins for the fp64 CPU oracle: each oracle function is checked against
something other than itself -- python-loop brute force, a library routine on a
special case, closed forms, invariants, the two-path equivalence the paper
states (Sec. 3.1) and the numbers the paper prints (Sec. 4, Sec. 5)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import synth

CANON = O.Dims(128, 8, 128, 512, 64)


def _tiny(h_q, g, d_h, r_kv, d_r, B, T, s_q, seed, dtype="f32", seqlens=None, d_v=0):
    w = synth.Workload("t", h_q, g, d_h, r_kv, d_r, batch=B, s_q=s_q, dtype=dtype, seed=seed, seqlen=T, d_v=d_v)
    x = synth.make_inputs(w, seqlens=seqlens)
    d = O.Dims(h_q, g, d_h, r_kv, d_r, d_v)
    f = {k: synth.to_f64(v) for k, v in x.items() if k not in ("seq_start", "seqlens")}
    return w, d, f, x["seq_start"].numpy(), x["seqlens"].numpy()


def _paths(d, f, ss, sl, s_q, scale):
    a = O.absorb_path(d, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, s_q, scale)
    g = O.gqa_path(d, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, s_q, scale)
    return a, g


# ---------------------------------------------------------------- integers


def test_group_map_values_and_repeat_equivalence():
    # hand-written values for the canonical config: 16 heads per group
    assert [O.group_of_head(CANON, i) for i in (0, 15, 16, 31, 32, 111, 112, 127)] == [0, 0, 1, 1, 2, 6, 7, 7]
    d = O.Dims(8, 2, 16, 32, 8)
    assert [O.group_of_head(d, i) for i in range(8)] == [0, 0, 0, 0, 1, 1, 1, 1]
    # Eq. (mqa) line 1: the per-head slices come from repeat(W, h_q/g)
    for h_q, g in ((128, 8), (32, 8), (8, 2), (28, 4), (20, 4), (6, 6), (5, 1)):
        dd = O.Dims(h_q, g, 4, 4, 2)
        rep = np.repeat(np.arange(g), h_q // g)
        assert [O.group_of_head(dd, i) for i in range(h_q)] == rep.tolist()


def test_visible_limit_values():
    # s_q = 1: the single query sees the whole cache, itself included
    assert O.visible_limit(4096, 1, 0) == 4096
    # s_q = 2: draft position 0 must not see draft position 1
    assert O.visible_limit(4096, 2, 0) == 4095
    assert O.visible_limit(4096, 2, 1) == 4096
    assert O.visible_limit(1, 2, 0) == 0 and O.visible_limit(1, 2, 1) == 1
    assert O.visible_limit(0, 2, 0) == 0 and O.visible_limit(0, 2, 1) == 0
    assert [O.visible_limit(10, 3, p) for p in range(3)] == [8, 9, 10]


def test_split_plan_values():
    assert O.split_plan(4096, 8) == [(512 * k, 512 * (k + 1)) for k in range(8)]
    assert O.split_plan(131072, 128)[-1] == (130048, 131072)
    # 100 tokens over 8 splits: ceil(100/8) = 13 -> one 64-token granule
    assert O.split_plan(100, 8) == [(0, 64), (64, 100)] + [(100, 100)] * 6
    assert O.split_plan(0, 4) == [(0, 0)] * 4
    assert O.split_plan(65, 1) == [(0, 65)]
    assert O.split_plan(4097, 2) == [(0, 2112), (2112, 4097)]
    rng = np.random.default_rng(1)
    for _ in range(200):
        T = int(rng.integers(0, 40000))
        S = int(rng.integers(1, 130))
        plan = O.split_plan(T, S)
        assert len(plan) == S and plan[0][0] == 0 and plan[-1][1] == T
        assert all(b <= e for b, e in plan)
        assert all(plan[k][1] == plan[k + 1][0] for k in range(S - 1))
        assert sum(e - b for b, e in plan) == T
        assert all(b % 64 == 0 for b, e in plan if e > b)


# ---------------------------------------------------------------- cache sizes and the printed Roofline numbers


def test_cache_sizes_printed_in_paper():
    assert O.mqa_cache_elems(CANON) == 576 and O.mqa_bytes(CANON, 1) == 1152
    assert O.gqa_cache_elems(CANON) == 2112 and O.gqa_bytes(CANON, 1) == 4224
    g4 = O.Dims(128, 4, 128, 512, 64)
    assert O.gqa_bytes(g4, 1) == 2176
    llama = O.Dims(32, 8, 128, 512, 64)
    assert O.mqa_cache_elems(llama) / (2 * llama.g * llama.d_h) * 100 == 28.125


def _golden(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "roofline_table.txt")) as fh:
        for line in fh:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_roofline_table_reproduced(golden_dir):
    rows = _golden(golden_dir)
    hw = {r[1]: (float(r[2]) * 1e12, float(r[3]) * 1e12, float(r[4])) for r in rows if r[0] == "hw"}
    for name, (peak, bw, ridge) in hw.items():
        assert abs(peak / bw - ridge) < 0.6
    L = 8192
    n_ops = 0
    for r in rows:
        if r[0] != "op":
            continue
        n_ops += 1
        _, gpu, path, g, s_q, cbytes, I, mem, cmp_, step, ktok = r
        g, s_q = int(g), int(s_q)
        d = O.Dims(128, g if path == "gqa" else 8, 128, 512, 64)
        if path == "mqa":
            nb, fl = O.mqa_bytes(d, L), O.mqa_flops(d, L, s_q)
        else:
            nb, fl = O.gqa_bytes(d, L), O.gqa_flops(d, L, s_q)
        assert nb // L == int(cbytes)
        assert abs(fl / nb - float(I)) <= 0.5  # printed as integers
        peak, bw, _ = hw[gpu]
        m, c, s = O.roofline_step(fl, nb, peak, bw)
        # printed to 2 decimals; allow one unit in the last place (30.83 vs 30.84, 9.07 vs 9.06)
        assert abs(m * 1e6 - float(mem)) <= 0.0101
        assert abs(c * 1e6 - float(cmp_)) <= 0.0101
        assert abs(s * 1e6 - float(step)) <= 0.0101
        # printed in whole K tok/s; 1/2.817us = 354.98K is printed as 354K, so allow one unit
        assert abs(s_q / s / 1e3 - float(ktok)) <= 1.0
    assert n_ops == 8
    for r in rows:
        if r[0] == "ai":
            _, path, g, s_q, val = r
            d = O.Dims(128, int(g), 128, 512, 64)
            if path == "mqa":
                ai = O.mqa_flops(d, L, int(s_q)) / O.mqa_bytes(d, L)
            else:
                ai = O.gqa_flops(d, L, int(s_q)) / O.gqa_bytes(d, L)
            # 484 is printed as twice the rounded 242 (exact value 483.6)
            assert abs(ai - float(val)) <= (0.5 if '.' not in val else 0.06)
        if r[0] == "mtp":
            peak, bw, _ = hw[r[1]]
            d = CANON
            s1 = O.roofline_step(O.mqa_flops(d, L, 1), O.mqa_bytes(d, L), peak, bw)[2]
            s2 = O.roofline_step(O.mqa_flops(d, L, 2), O.mqa_bytes(d, L), peak, bw)[2]
            assert abs(2 * s1 / s2 - float(r[2])) <= 0.006
    # bytes do not depend on s_q ("reads all L tokens once and reuses them across the s_q queries")
    assert O.mqa_bytes(CANON, L) == 2 * L * 576


# ---------------------------------------------------------------- contractions vs a library routine


def test_contractions_against_einsum_with_repeated_weights():
    w, d, f, ss, sl = _tiny(12, 3, 5, 7, 3, B=2, T=9, s_q=2, seed=5)
    rep_k = torch.from_numpy(np.repeat(f["w_uk"], d.hpg, axis=0))  # [h_q, r, d] : repeat(W, h_q/g)
    rep_v = torch.from_numpy(np.repeat(f["w_uv"], d.hpg, axis=0))
    qc, qr = torch.from_numpy(f["q_c"]), torch.from_numpy(f["q_r"])
    qh = O.absorb_q(d, f["q_c"], f["q_r"], f["w_uk"])
    ref = torch.cat([torch.einsum("bphd,hrd->bphr", qc, rep_k), qr], dim=-1).numpy()
    np.testing.assert_allclose(qh, ref, rtol=1e-13, atol=1e-13)
    oh = np.random.default_rng(0).standard_normal((2, 2, 12, 7))
    up = O.up_proj(d, oh, f["w_uv"])
    ref = torch.einsum("bphr,hrd->bphd", torch.from_numpy(oh), rep_v).numpy()
    np.testing.assert_allclose(up, ref, rtol=1e-13, atol=1e-13)
    kc, v, kr = O.expand_cache(d, f["cache"], f["w_uk"], f["w_uv"])
    c = torch.from_numpy(f["cache"])
    np.testing.assert_allclose(kc, torch.einsum("nr,grd->ngd", c[:, :7], torch.from_numpy(f["w_uk"])).numpy(),
                               rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(v, torch.einsum("nr,grd->ngd", c[:, :7], torch.from_numpy(f["w_uv"])).numpy(),
                               rtol=1e-13, atol=1e-13)
    np.testing.assert_array_equal(kr, f["cache"][:, 7:])
    assert kc.shape == (f["cache"].shape[0], 3, 5) and kr.shape[1] == 3


# ---------------------------------------------------------------- three evaluations agree


def test_c0_three_way_agreement():
    """Workload C0 (tiny check): both paths against each other and against brute force."""
    w = synth.WORKLOADS["C0"]
    x = synth.make_inputs(w)
    d = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    f = {k: synth.to_f64(v) for k, v in x.items() if k not in ("seq_start", "seqlens")}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    a, g = _paths(d, f, ss, sl, w.s_q, w.scale)
    bf = O.brute_force_path(d, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, w.s_q, w.scale)
    assert a.shape == (1, 1, 8, 16)
    scale_ref = np.abs(bf).max()
    assert np.abs(a - bf).max() <= 1e-12 * scale_ref
    assert np.abs(g - bf).max() <= 1e-12 * scale_ref
    assert np.abs(a - g).max() <= 1e-12 * scale_ref


@pytest.mark.parametrize("h_q,g,s_q", [(4, 1, 1), (4, 4, 2), (6, 2, 2), (6, 3, 3), (3, 1, 2)])
def test_random_tiny_three_way_agreement(h_q, g, s_q):
    # g = 1 is MQA, g = h_q is per-head MLA; ragged lengths including T < s_q
    seqlens = np.array([7, 1, 12], dtype=np.int32)
    w, d, f, ss, sl = _tiny(h_q, g, 4, 6, 2, B=3, T=0, s_q=s_q, seed=11 + h_q + g, seqlens=seqlens)
    a, gq = _paths(d, f, ss, sl, s_q, 0.4)
    bf = O.brute_force_path(d, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, s_q, 0.4)
    ref = max(np.abs(bf).max(), 1e-30)
    assert np.abs(a - bf).max() <= 1e-12 * ref
    assert np.abs(gq - bf).max() <= 1e-12 * ref


@pytest.mark.parametrize("d_h,d_v", [(4, 6), (6, 4), (3, 8)])
def test_separate_value_head_dim_three_way_agreement(d_h, d_v):
    """Sec. 3.2 "From MLA to GQLA": W~^UKV in R^{g (d_h + d_h^V) x r_kv} carries a value head dim of its own.
    Both paths against the python-loop brute force with d_v != d_h, plus the contractions against einsum."""
    seqlens = np.array([9, 2, 1], dtype=np.int32)
    w, d, f, ss, sl = _tiny(6, 2, d_h, 5, 2, B=3, T=0, s_q=2, seed=40 + d_h, seqlens=seqlens, d_v=d_v)
    assert f["w_uv"].shape == (2, 5, d_v) and f["w_uk"].shape == (2, 5, d_h)
    a, gq = _paths(d, f, ss, sl, 2, 0.37)
    bf = O.brute_force_path(d, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, 2, 0.37)
    assert a.shape == gq.shape == bf.shape == (3, 2, 6, d_v)
    ref = np.abs(bf).max()
    assert np.abs(a - bf).max() <= 1e-12 * ref and np.abs(gq - bf).max() <= 1e-12 * ref
    kc, v, kr = O.expand_cache(d, f["cache"], f["w_uk"], f["w_uv"])
    assert kc.shape[2] == d_h and v.shape[2] == d_v
    c = torch.from_numpy(f["cache"])
    np.testing.assert_allclose(v, torch.einsum("nr,grd->ngd", c[:, :5], torch.from_numpy(f["w_uv"])).numpy(),
                               rtol=1e-13, atol=1e-13)
    rep_v = torch.from_numpy(np.repeat(f["w_uv"], d.hpg, axis=0))
    oh = np.random.default_rng(1).standard_normal((3, 2, 6, 5))
    np.testing.assert_allclose(O.up_proj(d, oh, f["w_uv"]),
                               torch.einsum("bphr,hrd->bphd", torch.from_numpy(oh), rep_v).numpy(), rtol=1e-13, atol=1e-13)
    # cache elements per token: g (d_h + d_h^V) + d_h^R; equal value dim gives back 2 g d_h + d_h^R
    assert O.gqa_cache_elems(d) == 2 * (d_h + d_v) + 2
    assert O.gqa_cache_elems(O.Dims(128, 8, 128, 512, 64)) == 2112 == O.gqa_cache_elems(O.Dims(128, 8, 128, 512, 64, 128))
    assert O.gqa_flops(O.Dims(128, 8, 128, 512, 64, 128), 8192, 2) == O.gqa_flops(CANON, 8192, 2)


def test_two_paths_equal_at_larger_shapes():
    """Sec. 3.1 "Two equivalent decoding paths": same weights, same latent, same output."""
    for (h_q, g, T, s_q, seed) in ((16, 4, 300, 2, 1), (32, 8, 513, 1, 2), (8, 8, 129, 2, 3), (8, 1, 64, 1, 4)):
        w, d, f, ss, sl = _tiny(h_q, g, 32, 48, 16, B=2, T=T, s_q=s_q, seed=seed, dtype="bf16")
        a, gq = _paths(d, f, ss, sl, s_q, w.scale)
        assert np.abs(a - gq).max() <= 1e-10 * np.abs(a).max()


# ---------------------------------------------------------------- reduction to a library routine


def test_sparse_identity_weights_reduce_to_library_gqa():
    """Eq. (transgqla): with W^UK_j = W^UV_j the sparse identity selecting group j
    (r_kv = g d_h) the absorb path is ordinary GQA over the latent read as g K(=V)
    heads plus the shared RoPE key.  Ordinary GQA is torch's SDPA."""
    h_q, g, d_h, d_r, T, B, s_q = 8, 4, 6, 4, 37, 2, 2
    r_kv = g * d_h
    w, d, f, ss, sl = _tiny(h_q, g, d_h, r_kv, d_r, B=B, T=T, s_q=s_q, seed=21)
    W = np.zeros((g, r_kv, d_h))
    for j in range(g):
        for dd in range(d_h):
            W[j, j * d_h + dd, dd] = 1.0
    scale = 0.37
    mine = O.absorb_path(d, f["q_c"], f["q_r"], W, W, f["cache"], ss, sl, s_q, scale)
    mine_g = O.gqa_path(d, f["q_c"], f["q_r"], W, W, f["cache"], ss, sl, s_q, scale)
    cache = torch.from_numpy(f["cache"]).view(B, T, r_kv + d_r)
    lat = cache[..., :r_kv].view(B, T, g, d_h)
    k = torch.cat([lat, cache[..., r_kv:].unsqueeze(2).expand(B, T, g, d_r)], dim=-1)  # [B,T,g,d_h+d_r]
    k = k.repeat_interleave(h_q // g, dim=2).permute(0, 2, 1, 3)  # repeat_kv -> [B,h_q,T,D]
    v = lat.repeat_interleave(h_q // g, dim=2).permute(0, 2, 1, 3)
    q = torch.cat([torch.from_numpy(f["q_c"]), torch.from_numpy(f["q_r"])], dim=-1).permute(0, 2, 1, 3)
    mask = torch.ones(s_q, T, dtype=torch.bool)
    mask[0, T - 1] = False  # draft position 0 does not see draft position 1
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask, scale=scale)
    ref = ref.permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(mine, ref, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(mine_g, ref, rtol=1e-11, atol=1e-13)


def test_decode_kernels_against_library_sdpa_and_logsumexp():
    """decode_absorb is MQA over k_hat = [c; k_R], v_hat = c: one shared KV head."""
    w, d, f, ss, sl = _tiny(6, 2, 8, 10, 4, B=2, T=50, s_q=1, seed=8)
    qh = np.random.default_rng(3).standard_normal((2, 1, 6, 14))
    o, lse = O.decode_absorb(d, qh, f["cache"], ss, sl, 1, 0.3)
    c = torch.from_numpy(f["cache"]).view(2, 1, 50, 14)
    q = torch.from_numpy(qh).permute(0, 2, 1, 3)
    ref = torch.nn.functional.scaled_dot_product_attention(q, c.expand(2, 6, 50, 14), c[..., :10].expand(2, 6, 50, 10),
                                                           scale=0.3).permute(0, 2, 1, 3).numpy()
    np.testing.assert_allclose(o, ref, rtol=1e-11, atol=1e-13)
    x = 0.3 * torch.einsum("bhqd,bhkd->bhqk", q, c.expand(2, 6, 50, 14))
    np.testing.assert_allclose(lse, torch.logsumexp(x, dim=-1).permute(0, 2, 1).numpy(), rtol=1e-12)


# ---------------------------------------------------------------- softmax invariants and closed forms


def test_softmax_closed_forms():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((5, 7))
    K = rng.standard_normal((33, 7))
    V = rng.standard_normal((33, 3))
    o, lse = O._attend(q, K, V, 0.5, 0, 33)
    # weights sum to one: constant values come back unchanged
    Vc = np.tile(rng.standard_normal((1, 3)), (33, 1))
    oc, _ = O._attend(q, K, Vc, 0.5, 0, 33)
    np.testing.assert_allclose(oc, np.tile(Vc[:1], (5, 1)), rtol=1e-13)
    # a single key: output is its value, lse is its score
    o1, l1 = O._attend(q, K, V, 0.5, 4, 5)
    np.testing.assert_allclose(o1, np.tile(V[4:5], (5, 1)), rtol=1e-14)
    np.testing.assert_allclose(l1, 0.5 * q @ K[4], rtol=1e-13)
    # adding a constant c to every score leaves o alone and moves lse by c
    Kp = np.concatenate([K, np.ones((33, 1))], axis=1)
    qp = np.concatenate([q, np.full((5, 1), 3.25 / 0.5)], axis=1)
    o2, l2 = O._attend(qp, Kp, V, 0.5, 0, 33)
    np.testing.assert_allclose(o2, o, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(l2, lse + 3.25, rtol=1e-13)
    # two keys, hand-computed: scores 0 and ln 3 -> weights 1/4, 3/4
    o3, l3 = O._attend(np.array([[1.0]]), np.array([[0.0], [math.log(3.0)]]), np.array([[4.0], [8.0]]), 1.0, 0, 2)
    assert abs(o3[0, 0] - 7.0) < 1e-14 and abs(l3[0] - math.log(4.0)) < 1e-14
    # huge scores do not overflow
    o4, l4 = O._attend(np.array([[1000.0]]), np.array([[1.0], [1.0]]), np.array([[1.0], [3.0]]), 1.0, 0, 2)
    assert abs(o4[0, 0] - 2.0) < 1e-14 and abs(l4[0] - (1000.0 + math.log(2.0))) < 1e-10
    # empty range
    o5, l5 = O._attend(q, K, V, 0.5, 6, 6)
    assert (o5 == 0).all() and np.isneginf(l5).all()


# ---------------------------------------------------------------- causal MTP mask


@pytest.mark.parametrize("path", ["absorb", "gqa"])
def test_mtp_mask_equals_two_single_steps(path):
    """s_q = 2 at length T == s_q = 1 at T-1 (row 0) and at T (row 1), up to the
    BLAS's shape-dependent summation order."""
    T = 77
    w, d, f, ss, sl = _tiny(8, 2, 8, 12, 4, B=2, T=T, s_q=2, seed=31)
    fn = O.absorb_path if path == "absorb" else O.gqa_path
    two = fn(d, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, 2, 0.3)
    for p, Tp in ((0, T - 1), (1, T)):
        one = fn(d, f["q_c"][:, p:p + 1], f["q_r"][:, p:p + 1], f["w_uk"], f["w_uv"], f["cache"], ss,
                 np.full((2,), Tp, dtype=np.int32), 1, 0.3)
        np.testing.assert_allclose(two[:, p], one[:, 0], rtol=1e-12, atol=1e-15)


def test_rows_without_visible_keys():
    seqlens = np.array([1, 0, 2], dtype=np.int32)
    w, d, f, ss, sl = _tiny(4, 2, 4, 6, 2, B=3, T=0, s_q=2, seed=41, seqlens=seqlens)
    qh = O.absorb_q(d, f["q_c"], f["q_r"], f["w_uk"])
    o, lse = O.decode_absorb(d, qh, f["cache"], ss, sl, 2, 0.5)
    assert (o[0, 0] == 0).all() and np.isneginf(lse[0, 0]).all()  # T=1: draft 0 sees nothing
    np.testing.assert_allclose(o[0, 1], np.tile(f["cache"][0, :6], (4, 1)), rtol=1e-14)  # draft 1 sees row 0 only
    assert (o[1] == 0).all() and np.isneginf(lse[1]).all()  # T=0
    assert np.isfinite(lse[2]).all()


# ---------------------------------------------------------------- split-KV + combine


@pytest.mark.parametrize("path", ["absorb", "gqa"])
def test_split_combine_invariance(path):
    seqlens = np.array([1000, 63, 129, 2], dtype=np.int32)
    w, d, f, ss, sl = _tiny(8, 4, 8, 16, 4, B=4, T=0, s_q=2, seed=51, dtype="bf16", seqlens=seqlens)
    if path == "absorb":
        q = O.absorb_q(d, f["q_c"], f["q_r"], f["w_uk"])
        part = lambda S: O.decode_absorb_partials(d, q, f["cache"], ss, sl, 2, 0.25, S)
    else:
        kc, v, kr = O.expand_cache(d, f["cache"], f["w_uk"], f["w_uv"])
        q = np.concatenate([f["q_c"], f["q_r"]], axis=-1)
        part = lambda S: O.decode_gqa_partials(d, q, kc, v, kr, ss, sl, 2, 0.25, S)
    o1, l1 = O.combine_splits(*part(1))
    for S in (8, 32, 128):
        op, lp = part(S)
        assert op.shape[1] == S
        # splits beyond the sequence are empty: zero partial, -inf lse
        assert np.isneginf(lp[1, 1:]).all() and (op[1, 1:] == 0).all()
        oS, lS = O.combine_splits(op, lp)
        np.testing.assert_allclose(oS, o1, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(lS, l1, rtol=1e-12)


def test_combine_closed_form_and_dead_rows():
    # two splits with lse = ln 1 and ln 3: weights 1/4 and 3/4
    o_part = np.array([[[[2.0]], [[6.0]]]]).reshape(1, 2, 1, 1)
    lse_part = np.array([[[0.0], [math.log(3.0)]]]).reshape(1, 2, 1)
    o, l = O.combine_splits(o_part, lse_part)
    assert abs(o[0, 0, 0] - 5.0) < 1e-14 and abs(l[0, 0] - math.log(4.0)) < 1e-14
    # an empty split is ignored; all-empty rows give 0 and -inf without NaN
    o_part = np.array([1.0, 0.0, 0.0, 0.0]).reshape(2, 2, 1, 1)
    lse_part = np.array([0.5, -np.inf, -np.inf, -np.inf]).reshape(2, 2, 1)
    o, l = O.combine_splits(o_part, lse_part)
    assert o[0, 0, 0] == 1.0 and l[0, 0] == 0.5
    assert o[1, 0, 0] == 0.0 and np.isneginf(l[1, 0]) and not np.isnan(o).any()


def test_balanced_plan_invariants():
    """Pins of the oracle's balanced split plan that follow from its definition alone: the pieces of a
    sequence are disjoint, ordered, cover exactly [0, T), start on 128-row tile boundaries and are at
    most S; with one worker nothing is cut; a uniform batch on as many workers as sequences is not cut
    either; hand-worked case: T = (300, 100, 0, 260) rows = (3, 1, 0, 3) tiles on 3 workers, S = 3 ->
    share 3: worker 0 gets sequence 0, worker 1 sequence 1 and tiles 0-1 of sequence 3, worker 2 its tile 2."""
    rng = np.random.default_rng(5)
    for _ in range(200):
        n = int(rng.integers(1, 30))
        sl = [int(x) for x in rng.integers(0, 20000, size=n)]
        S, W = int(rng.integers(2, 7)), int(rng.integers(1, 100))
        plans = O.balanced_plan(sl, S, W)
        assert len(plans) == n
        for T, plan in zip(sl, plans):
            assert len(plan) == S
            live = [(lo, hi) for lo, hi in plan if hi > lo]
            assert plan[:len(live)] == live and all(pc == (0, 0) for pc in plan[len(live):])
            pos = 0
            for lo, hi in live:
                assert lo == pos and lo % 128 == 0
                pos = hi
            assert pos == T
    assert O.balanced_plan([4096] * 8, 2, 1) == [[(0, 4096), (0, 0)]] * 8
    assert O.balanced_plan([4096] * 8, 2, 8) == [[(0, 4096), (0, 0)]] * 8
    assert O.balanced_plan([300, 100, 0, 260], 3, 3) == [
        [(0, 300), (0, 0), (0, 0)], [(0, 100), (0, 0), (0, 0)], [(0, 0)] * 3, [(0, 256), (256, 260), (0, 0)]]


def test_partials_with_an_explicit_plan_combine_to_the_same_output():
    """Any partition of the rows gives the same attention output after the LSE merge (fp64)."""
    w = synth.Workload("bp", 8, 2, 16, 32, 8, batch=3, s_q=2, dtype="f32", seed=21)
    x = synth.make_inputs(w, seqlens=np.array([300, 0, 517], dtype=np.int32), q_gain=3.0)
    f = {k: synth.to_f64(v) for k, v in x.items() if k not in ("seq_start", "seqlens")}
    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    qh = O.absorb_q(od, f["q_c"], f["q_r"], f["w_uk"])
    ref, ref_lse = O.combine_splits(*O.decode_absorb_partials(od, qh, f["cache"], ss, sl, w.s_q, w.scale, 1))
    for S, W in ((2, 3), (3, 2), (4, 7)):
        plans = O.balanced_plan([int(t) for t in sl], S, W)
        o, lse = O.combine_splits(*O.decode_absorb_partials(od, qh, f["cache"], ss, sl, w.s_q, w.scale, S, plans))
        np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)
        fin = np.isfinite(ref_lse)
        assert np.array_equal(np.isneginf(lse), np.isneginf(ref_lse))
        np.testing.assert_allclose(lse[fin], ref_lse[fin], rtol=1e-12, atol=1e-12)


def test_unpage_inverts_the_paged_layout():
    """Paging is storage only.  The scatter that builds a paged pool (the input generator) and the oracle's
    gather are written independently; composed, they must give back the packed rows, for page sizes that do
    and do not divide the lengths, with empty sequences, and with the pages in a shuffled order."""
    rng = np.random.default_rng(5)
    seqlens = np.array([37, 0, 128, 1, 300], dtype=np.int32)
    seq_start = np.concatenate([[0], np.cumsum(seqlens)[:-1]]).astype(np.int64)
    packed = torch.from_numpy(rng.standard_normal((int(seqlens.sum()), 6)).astype(np.float32))
    for page_size in (1, 16, 128, 256):
        paged, table = synth.to_paged(packed, seq_start, seqlens, page_size, seed=11)
        assert paged.shape[0] % page_size == 0
        back, ss = O.unpage(paged.numpy(), table.numpy(), page_size, seqlens)
        assert np.array_equal(ss, seq_start)
        assert np.array_equal(back, packed.numpy())
    # the identity table on an already paged-shaped array is a no-op
    ident = np.arange(4, dtype=np.int32).reshape(1, 4)
    x = rng.standard_normal((64, 3))
    back, _ = O.unpage(x, ident, 16, np.array([64], dtype=np.int32))
    assert np.array_equal(back, x)
