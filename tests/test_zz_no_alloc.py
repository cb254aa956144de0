"""gqla_decode_gqa_noalloc: the GQA-path step for hosts that cannot allocate device memory while
decoding (a server that handed the whole GPU to its own memory manager, a loop that cannot take the
device-wide stall of cudaMalloc, a bare C caller).  It keeps the split partials in an array built
into the library instead of in caller buffers, so it must give what gqla_decode_gqa followed by
gqla_combine_splits gives on caller buffers -- also on a second call, when the array still holds
the first call's partials.

This file is named so that pytest collects it after every other test file."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import binding as B
from paper_2605_15250_b200 import build as gbuild
from paper_2605_15250_b200 import synth

REL, ABS = 1e-2, 1e-3  # the tolerance of the parity tests


def test_noalloc_rejects_calls_beyond_its_capacity():
    """More partial rows than the built-in array holds: a capacity error, and nothing is launched
    (the pointers here are never dereferenced)."""
    gbuild.build()
    L = B.lib()
    d = B.make_dims(128, 8, 128, 512, 64)
    p = ctypes.c_void_p(0x1000)
    r = ctypes.byref
    # 64 sequences x 8 splits x 2 queries x 128 heads = 131072 rows > 65536
    assert L.gqla_decode_gqa_noalloc(r(d), 0, 64, 2, 0.1, 8, p, p, p, p, 64, 10, p, p, p, None, None, None) == 8
    # 65536 rows fit the row limit but 65536 x 128 floats exceed the 4 Mi float limit
    assert L.gqla_decode_gqa_noalloc(r(d), 0, 64, 2, 0.1, 4, p, p, p, p, 64, 10, p, p, p, None, None, None) == 8
    assert "capacity" in L.gqla_status_str(8).decode()
    assert L.gqla_decode_gqa_noalloc(r(d), 0, 1, 1, 0.1, 1, p, p, p, p, 64, 10, p, p, None, None, None, None) == 1


@pytest.mark.gpu
def test_noalloc_matches_caller_buffer_path_twice_in_a_row():
    gbuild.build()
    assert torch.cuda.is_available()
    B.lib()
    B.set_policy(B.POLICY_AUTO)
    w = synth.Workload("noalloc", 128, 8, 128, 512, 64, batch=4, s_q=2, dtype="bf16", seed=0x2A)
    seqlens = np.array([700, 1, 129, 2050], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=4.0)
    dims = B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    cache, ss, sl = x["cache"].cuda(), x["seq_start"].cuda(), x["seqlens"].cuda()
    N = cache.shape[0]
    k_c = torch.empty((N, w.g, w.d_h), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k_c)
    B.gqla_expand_cache(dims, cache, x["w_uk"].cuda(), x["w_uv"].cuda(), k_c, v, None)
    k_r = cache[:, w.r_kv:]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    q_first = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
    q_second = (-0.5 * q_first.float()).flip(2).contiguous().to(torch.bfloat16)
    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    f_kc, f_v, f_kr = synth.to_f64(k_c), synth.to_f64(v), synth.to_f64(k_r)

    # second call: other queries and another split count, so stale partials of the first call would show
    for q, S in ((q_first, 3), (q_second, 2)):
        o_part = torch.empty((w.batch, S, w.s_q, w.h_q, w.d_h), dtype=torch.float32, device="cuda")
        lse_part = torch.empty((w.batch, S, w.s_q, w.h_q), dtype=torch.float32, device="cuda")
        ref = torch.empty((w.batch, w.s_q, w.h_q, w.d_h), dtype=torch.bfloat16, device="cuda")
        ref_lse = torch.empty((w.batch, w.s_q, w.h_q), dtype=torch.float32, device="cuda")
        B.gqla_decode_gqa(dims, q, k_c, v, k_r, ss, sl, w.scale, S, o_part, lse_part, status)
        B.gqla_combine_splits(o_part, lse_part, ref, ref_lse)

        out = torch.full_like(ref, float("nan"))
        lse = torch.full_like(ref_lse, float("nan"))
        B.gqla_decode_gqa_noalloc(dims, q, k_c, v, k_r, ss, sl, w.scale, S, out, lse, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0

        got, want = out.float().cpu().numpy(), ref.float().cpu().numpy()
        assert not np.isnan(got).any()
        bound = REL * np.abs(want).max() + ABS
        assert np.abs(got - want).max() <= bound, (S, np.abs(got - want).max(), bound)
        gl, wl = lse.cpu().numpy(), ref_lse.cpu().numpy()
        assert np.array_equal(np.isneginf(gl), np.isneginf(wl))
        fin = ~np.isneginf(wl)
        assert np.abs(gl[fin] - wl[fin]).max() <= REL * np.abs(wl[fin]).max() + ABS
        # and against the CPU checker on the very planes the kernel read
        o_ref, l_ref = O.decode_gqa(od, synth.to_f64(q), f_kc, f_v, f_kr, x["seq_start"].numpy(), x["seqlens"].numpy(),
                                    w.s_q, w.scale)
        assert np.abs(got - o_ref).max() <= REL * np.abs(o_ref).max() + ABS
        assert np.array_equal(np.isneginf(gl), np.isneginf(l_ref))
        assert np.abs(gl[fin] - l_ref[fin]).max() <= REL * np.abs(l_ref[fin]).max() + ABS


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,policy", [("f32", "auto"), ("bf16", "generic")])
def test_noalloc_other_kernels_and_types(dtype, policy):
    """The fp32 storage type and the generic kernel policy go through the same built-in array; an empty
    call first, as a host would make at start-up to have the array placed."""
    gbuild.build()
    assert torch.cuda.is_available()
    B.lib()
    B.set_policy(B.POLICY_GENERIC if policy == "generic" else B.POLICY_AUTO)
    try:
        w = synth.Workload("noalloc2", 8, 2, 16, 32, 8, batch=3, s_q=2, dtype=dtype, seed=0x2B)
        seqlens = np.array([70, 0, 131], dtype=np.int32)
        x = synth.make_inputs(w, seqlens=seqlens, q_gain=2.0)
        dims = B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
        od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
        f = {k: synth.to_f64(t) for k, t in x.items() if k not in ("seq_start", "seqlens")}
        kc_ref, v_ref, kr_ref = O.expand_cache(od, f["cache"], f["w_uk"], f["w_uv"])
        td = torch.bfloat16 if dtype == "bf16" else torch.float32
        k_c, v, k_r = (torch.from_numpy(np.ascontiguousarray(a)).to(td).cuda() for a in (kc_ref, v_ref, kr_ref))
        q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
        ss, sl = x["seq_start"].cuda(), x["seqlens"].cuda()
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        out = torch.full((w.batch, w.s_q, w.h_q, w.d_h), float("nan"), dtype=td, device="cuda")
        lse = torch.full((w.batch, w.s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
        # warm-up: an empty batch (B = 0) performs the address query and launches nothing
        B.gqla_decode_gqa_noalloc(dims, q[:0], k_c, v, k_r, ss[:0], sl[:0], w.scale, 1, out, None, status)
        assert torch.isnan(out.float()).all()
        o_ref, l_ref = O.decode_gqa(od, synth.to_f64(q), synth.to_f64(k_c), synth.to_f64(v), synth.to_f64(k_r),
                                    x["seq_start"].numpy(), x["seqlens"].numpy(), w.s_q, w.scale)
        for S in (2, 1):
            out.fill_(float("nan")); lse.fill_(float("nan"))
            B.gqla_decode_gqa_noalloc(dims, q, k_c, v, k_r, ss, sl, w.scale, S, out, lse, status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            got, gl = out.float().cpu().numpy(), lse.cpu().numpy()
            assert not np.isnan(got).any()
            assert np.abs(got - o_ref).max() <= REL * np.abs(o_ref).max() + ABS
            assert np.array_equal(np.isneginf(gl), np.isneginf(l_ref))
            fin = ~np.isneginf(l_ref)
            assert np.abs(gl[fin] - l_ref[fin]).max() <= REL * np.abs(l_ref[fin]).max() + ABS
    finally:
        B.set_policy(B.POLICY_AUTO)
