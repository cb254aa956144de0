"""FP8 (E4M3) cache: the library's quantisers must produce the oracle's codes bit for bit (the rounding decision is
taken in fp32 on both sides), and both decode paths over the quantised cache must match the oracle's plain
attention on the decoded numbers."""
import numpy as np
import pytest
import torch

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import binding as B
from paper_2605_15250_b200 import build as gbuild
from paper_2605_15250_b200 import synth
from tests.parity_util import assert_close

pytestmark = pytest.mark.gpu

# Tolerance of the FP8 decode calls against the oracle on the same codes.  The generic kernels keep the
# probabilities in fp32: the bf16-path tolerance applies.  The tensor-core kernels round them to E4M3 (4
# significant bits, unit roundoff u = 2^-4) before P.V: |err| <= u sum_s p_s |v_s - o| / sum_s p_s, i.e. at most
# 2u max|v| and typically u / sqrt(3) times the spread of the values under the softmax weights.
REL_TC, ABS_TC = 6e-2, 4e-3


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gbuild.build()
    assert torch.cuda.is_available()
    B.lib()
    yield
    B.set_policy(B.POLICY_AUTO)


def _scales(t: torch.Tensor, split: int):
    a = float(t[..., :split].abs().max()) / 448.0
    b = float(t[..., split:].abs().max()) / 448.0 if split < t.shape[-1] else a
    return max(a, 1e-8), max(b, 1e-8)


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_quantisers_give_the_oracle_codes_bit_for_bit(dtype):
    rng = np.random.default_rng(9)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    x = torch.from_numpy((rng.standard_normal((301, 577)) * rng.choice([1e-3, 1.0, 30.0], size=(301, 1))).astype(np.float32)).to(td)
    x[5] = 0
    x[7, 3] = 1e6   # saturates
    xs = x[:, :576]  # strided rows (stride 577), width 576
    sa, sb = 0.0371, 0.0113
    dst = torch.empty((301, 576), dtype=torch.uint8, device="cuda")
    B.gqla_quantize_cols_e4m3(xs.cuda(), 512, sa, sb, dst)
    ref = O.quantize_cols_e4m3(xs.float().numpy(), 512, sa, sb)
    got = dst.cpu().numpy()
    same = (got == ref) | (((got & 0x7F) == 0) & ((ref & 0x7F) == 0))  # the sign of a zero is immaterial
    assert same.all(), np.argwhere(~same)[:5]
    q = x[:, :576].contiguous().view(7, 43, 576)
    d8 = torch.empty(q.shape, dtype=torch.uint8, device="cuda")
    rs = torch.empty(q.shape[:-1], dtype=torch.float32, device="cuda")
    B.gqla_quantize_rows_e4m3(q.cuda(), 512, sa, sb, d8, rs)
    c_ref, s_ref = O.quantize_rows_e4m3(q.float().numpy(), 512, sa, sb)
    assert np.array_equal(rs.cpu().numpy(), s_ref)
    got = d8.cpu().numpy()
    same = (got == c_ref) | (((got & 0x7F) == 0) & ((c_ref & 0x7F) == 0))
    assert same.all(), np.argwhere(~same)[:5]


@pytest.mark.parametrize("dims,policy", [(dict(h_q=8, g=2, d_h=16, r_kv=32, d_r=8), "auto"),
                                         (dict(h_q=128, g=8, d_h=128, r_kv=512, d_r=64), "generic"),
                                         (dict(h_q=128, g=8, d_h=128, r_kv=512, d_r=64), "auto"),
                                         (dict(h_q=32, g=8, d_h=128, r_kv=512, d_r=64), "auto")])
@pytest.mark.parametrize("s_q", [1, 2])
def test_fp8_decode_both_paths(dims, policy, s_q):
    B.set_policy(B.POLICY_GENERIC if policy == "generic" else B.POLICY_AUTO)
    w = synth.Workload("f8", batch=3, s_q=s_q, dtype="bf16", seed=31, **dims)
    seqlens = np.array([700, 1, 385], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=3.0)
    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    bd = B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    dev = {k: t.cuda() for k, t in x.items()}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    N, Bn, S = x["cache"].shape[0], w.batch, 2
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    tc = policy == "auto" and dims["d_h"] == 128
    rel, abs_ = (REL_TC, ABS_TC) if tc else (1e-2, 1e-3)

    # ---- absorb path: quantise the latent cache and q_hat, attend, compare with the oracle on the same codes
    sc, sr = _scales(x["cache"].float(), w.r_kv)
    cache8 = torch.empty((N, w.d_abs), dtype=torch.uint8, device="cuda")
    B.gqla_quantize_cols_e4m3(dev["cache"], w.r_kv, sc, sr, cache8)
    q_hat = torch.empty((Bn, s_q, w.h_q, w.d_abs), dtype=torch.bfloat16, device="cuda")
    B.gqla_absorb_q(bd, dev["q_c"], dev["q_r"], dev["w_uk"], q_hat)
    q8 = torch.empty(q_hat.shape, dtype=torch.uint8, device="cuda")
    qs = torch.empty(q_hat.shape[:-1], dtype=torch.float32, device="cuda")
    B.gqla_quantize_rows_e4m3(q_hat, w.r_kv, sc, sr, q8, qs)
    o_part = torch.full((Bn, S, s_q, w.h_q, w.r_kv), float("nan"), dtype=torch.float32, device="cuda")
    lse_part = torch.full((Bn, S, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    B.gqla_decode_absorb_fp8(bd, q8, qs, cache8, sc, dev["seq_start"], dev["seqlens"], w.scale, S, o_part, lse_part, status)
    op_ref, lp_ref = O.decode_absorb_fp8_partials(od, q8.cpu().numpy(), qs.cpu().numpy(), cache8.cpu().numpy(), sc, ss, sl,
                                                  s_q, w.scale, S)
    assert_close(o_part.cpu().numpy(), op_ref, "decode_absorb_fp8 o_part", rel, abs_)
    assert_close(lse_part.cpu().numpy(), lp_ref, "decode_absorb_fp8 lse_part", 1e-2, 1e-3)

    if tc:  # the whole-sequence call: bf16 o_hat in one pass (tensor-core shapes only)
        o_hat = torch.full((Bn, s_q, w.h_q, w.r_kv), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((Bn, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
        B.gqla_decode_absorb_fp8_final(bd, q8, qs, cache8, sc, dev["seq_start"], dev["seqlens"], w.scale, o_hat, lse, status)
        o1, l1 = O.decode_absorb_fp8_partials(od, q8.cpu().numpy(), qs.cpu().numpy(), cache8.cpu().numpy(), sc, ss, sl, s_q,
                                              w.scale, 1)
        assert_close(o_hat.float().cpu().numpy(), o1[:, 0], "decode_absorb_fp8_final o_hat", rel, abs_)
        assert_close(lse.cpu().numpy(), l1[:, 0], "decode_absorb_fp8_final lse", 1e-2, 1e-3)

    # ---- GQA path: expand in bf16, quantise the three planes and q, attend
    k_c = torch.empty((N, w.g, w.d_h), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k_c)
    B.gqla_expand_cache(bd, dev["cache"], dev["w_uk"], dev["w_uv"], k_c, v, None)
    sk, _ = _scales(k_c.float(), w.d_h)
    sv, _ = _scales(v.float(), w.d_h)
    kc8 = torch.empty(k_c.shape, dtype=torch.uint8, device="cuda")
    v8 = torch.empty(v.shape, dtype=torch.uint8, device="cuda")
    kr8 = torch.empty((N, w.d_r), dtype=torch.uint8, device="cuda")
    B.gqla_quantize_cols_e4m3(k_c, w.d_h, sk, sk, kc8)
    B.gqla_quantize_cols_e4m3(v, w.d_h, sv, sv, v8)
    B.gqla_quantize_cols_e4m3(dev["cache"][:, w.r_kv:], w.d_r, sr, sr, kr8)
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
    q8g = torch.empty(q.shape, dtype=torch.uint8, device="cuda")
    qsg = torch.empty(q.shape[:-1], dtype=torch.float32, device="cuda")
    B.gqla_quantize_rows_e4m3(q, w.d_h, sk, sr, q8g, qsg)
    og_part = torch.full((Bn, S, s_q, w.h_q, w.d_h), float("nan"), dtype=torch.float32, device="cuda")
    lg_part = torch.full((Bn, S, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    B.gqla_decode_gqa_fp8(bd, q8g, qsg, kc8, v8, kr8, sv, dev["seq_start"], dev["seqlens"], w.scale, S, og_part, lg_part, status)
    og_ref, lg_ref = O.decode_gqa_fp8_partials(od, q8g.cpu().numpy(), qsg.cpu().numpy(), kc8.cpu().numpy(), v8.cpu().numpy(),
                                               kr8.cpu().numpy(), sv, ss, sl, s_q, w.scale, S)
    assert_close(og_part.cpu().numpy(), og_ref, "decode_gqa_fp8 o_part", rel, abs_)
    assert_close(lg_part.cpu().numpy(), lg_ref, "decode_gqa_fp8 lse_part", 1e-2, 1e-3)
    assert int(status.item()) == 0

    # the two quantised paths still describe the same attention: against the unquantised oracle within the input
    # rounding (two E4M3 roundings per product in the scores, one per value)
    ref = O.decode_gqa_partials(od, synth.to_f64(q), synth.to_f64(k_c), synth.to_f64(v), synth.to_f64(dev["cache"][:, w.r_kv:]),
                                ss, sl, s_q, w.scale, S)[0]
    assert np.abs(og_part.cpu().numpy() - ref).max() <= 0.3 * np.abs(ref).max()

    # ---- the balanced plan (num_splits < 0) cuts the sequences differently; what it must reproduce is the merged
    # attention output, which no plan changes: both calls, merged, against the oracle's merged partials
    o_ref, l_ref = O.combine_splits(op_ref, lp_ref)
    g_ref, gl_ref = O.combine_splits(og_ref, lg_ref)
    for slots in (2, 4):
        o_part = torch.full((Bn, slots, s_q, w.h_q, w.r_kv), float("nan"), dtype=torch.float32, device="cuda")
        lse_part = torch.full((Bn, slots, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
        B.gqla_decode_absorb_fp8(bd, q8, qs, cache8, sc, dev["seq_start"], dev["seqlens"], w.scale, -slots, o_part, lse_part,
                                 status)
        o_m = torch.empty((Bn, s_q, w.h_q, w.r_kv), dtype=torch.float32, device="cuda")
        l_m = torch.empty((Bn, s_q, w.h_q), dtype=torch.float32, device="cuda")
        B.gqla_combine_splits(o_part, lse_part, o_m, l_m)
        assert_close(o_m.cpu().numpy(), o_ref, "balanced decode_absorb_fp8, merged", rel, abs_)
        assert_close(l_m.cpu().numpy(), l_ref, "balanced decode_absorb_fp8, merged lse", 1e-2, 1e-3)
        og_part = torch.full((Bn, slots, s_q, w.h_q, w.d_h), float("nan"), dtype=torch.float32, device="cuda")
        lg_part = torch.full((Bn, slots, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
        B.gqla_decode_gqa_fp8(bd, q8g, qsg, kc8, v8, kr8, sv, dev["seq_start"], dev["seqlens"], w.scale, -slots, og_part,
                              lg_part, status)
        g_m = torch.empty((Bn, s_q, w.h_q, w.d_h), dtype=torch.float32, device="cuda")
        gl_m = torch.empty((Bn, s_q, w.h_q), dtype=torch.float32, device="cuda")
        B.gqla_combine_splits(og_part, lg_part, g_m, gl_m)
        assert_close(g_m.cpu().numpy(), g_ref, "balanced decode_gqa_fp8, merged", rel, abs_)
        assert_close(gl_m.cpu().numpy(), gl_ref, "balanced decode_gqa_fp8, merged lse", 1e-2, 1e-3)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
