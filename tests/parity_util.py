"""Helpers shared by the GPU parity tests: run the CUDA library and the fp64 oracle on
the same seeded inputs and compare element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import binding as B
from paper_2605_15250_b200 import synth
from paper_2605_15250_b200.decoder import GqlaDecoder

# Tolerance fixed by the benchmark spec for bf16 inputs with fp32 accumulation.
REL, ABS = 1e-2, 1e-3


def assert_close(got, ref, what: str, rel: float = REL, abs_: float = ABS) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    inf_ref = np.isneginf(ref)
    assert np.array_equal(np.isneginf(got), inf_ref), f"{what}: -inf pattern differs"
    assert not np.isnan(got).any(), f"{what}: NaN in output"
    fin = ~inf_ref
    if not fin.any():
        return 0.0
    bound = rel * np.abs(ref[fin]).max() + abs_
    err = np.abs(got[fin] - ref[fin]).max()
    assert err <= bound, f"{what}: max|err| {err:.3e} > {bound:.3e} (max|ref| {np.abs(ref[fin]).max():.3e})"
    return float(err)


class Canaried:
    """A device tensor with guard regions before and behind it (the pool offers no compute-sanitizer): `t` is the
    tensor a kernel writes, check() fails if a single guard byte has changed."""

    PAD = 4096  # bytes on each side
    BYTE = 0xA5

    def __init__(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((self.PAD + n + self.PAD,), self.BYTE, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.PAD:self.PAD + n].view(dtype).view(*shape)
        self.n = n

    def check(self, what: str) -> None:
        head, tail = self.raw[:self.PAD], self.raw[self.PAD + self.n:]
        assert bool((head == self.BYTE).all()) and bool((tail == self.BYTE).all()), f"{what}: wrote outside its buffer"


def dims_of(w: synth.Workload):
    return O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r), B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)


def tdtype(w: synth.Workload):
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def round_to(w: synth.Workload, a: np.ndarray) -> torch.Tensor:
    """fp64 array -> storage dtype (round to nearest even), on the CPU."""
    return torch.from_numpy(np.ascontiguousarray(a)).to(tdtype(w))


def stagewise(w: synth.Workload, seqlens, num_splits: int, q_gain: float = 1.0, check_partials: bool = True):
    """Runs every library call on its own, each fed the oracle's (storage-rounded) output of the
    stage before, and compares with the oracle on the same inputs.  Returns max errors."""
    od, bd = dims_of(w)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=q_gain)
    dev = {k: v.cuda() for k, v in x.items()}
    f = {k: synth.to_f64(v) for k, v in x.items() if k not in ("seq_start", "seqlens")}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    Bn, s_q, S = w.batch, w.s_q, num_splits
    dt = tdtype(w)
    errs = {}
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    # absorb_q
    q_hat = torch.empty((Bn, s_q, w.h_q, w.d_abs), dtype=dt, device="cuda")
    B.gqla_absorb_q(bd, dev["q_c"], dev["q_r"], dev["w_uk"], q_hat)
    qh_ref = O.absorb_q(od, f["q_c"], f["q_r"], f["w_uk"])
    errs["absorb_q"] = assert_close(q_hat.float().cpu().numpy(), qh_ref, "absorb_q")

    # decode_absorb on the oracle's q_hat rounded to storage
    qh_in = round_to(w, qh_ref)
    o_part = torch.full((Bn, S, s_q, w.h_q, w.r_kv), float("nan"), dtype=torch.float32, device="cuda")
    lse_part = torch.full((Bn, S, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    B.gqla_decode_absorb(bd, qh_in.cuda(), dev["cache"], dev["seq_start"], dev["seqlens"], w.scale, S, o_part,
                         lse_part, status)
    op_ref, lp_ref = O.decode_absorb_partials(od, synth.to_f64(qh_in), f["cache"], ss, sl, s_q, w.scale, S)
    if check_partials:
        errs["absorb_o_part"] = assert_close(o_part.cpu().numpy(), op_ref, "decode_absorb o_part")
        errs["absorb_lse_part"] = assert_close(lse_part.cpu().numpy(), lp_ref, "decode_absorb lse_part")

    # the whole-sequence call: final latent output in the storage dtype, no partials
    oh_w = torch.full((Bn, s_q, w.h_q, w.r_kv), float("nan"), dtype=dt, device="cuda")
    lse_w = torch.full((Bn, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    B.gqla_decode_absorb_final(bd, qh_in.cuda(), dev["cache"], dev["seq_start"], dev["seqlens"], w.scale, oh_w, lse_w, status)
    ohw_ref, lw_ref = O.decode_absorb(od, synth.to_f64(qh_in), f["cache"], ss, sl, s_q, w.scale)
    errs["absorb_final_o"] = assert_close(oh_w.float().cpu().numpy(), ohw_ref, "decode_absorb_final o_hat")
    errs["absorb_final_lse"] = assert_close(lse_w.cpu().numpy(), lw_ref, "decode_absorb_final lse")
    oh_n = torch.full_like(oh_w, float("nan"))
    B.gqla_decode_absorb_final(bd, qh_in.cuda(), dev["cache"], dev["seq_start"], dev["seqlens"], w.scale, oh_n, None, status)
    assert torch.equal(oh_n, oh_w), "decode_absorb_final without an lse output must give the same o_hat"

    # combine on the oracle's partials (fp32)
    op_in = torch.from_numpy(op_ref).float()
    lp_in = torch.from_numpy(lp_ref).float()
    o_hat = torch.empty((Bn, s_q, w.h_q, w.r_kv), dtype=dt, device="cuda")
    lse = torch.empty((Bn, s_q, w.h_q), dtype=torch.float32, device="cuda")
    B.gqla_combine_splits(op_in.cuda(), lp_in.cuda(), o_hat, lse)
    oh_ref, l_ref = O.combine_splits(op_in.double().numpy(), lp_in.double().numpy())
    errs["combine_o"] = assert_close(o_hat.float().cpu().numpy(), oh_ref, "combine o")
    errs["combine_lse"] = assert_close(lse.cpu().numpy(), l_ref, "combine lse")

    # combine fused with up_proj, on the same partials, against the unrounded composition
    o_f = torch.empty((Bn, s_q, w.h_q, w.d_h), dtype=dt, device="cuda")
    lse_f = torch.empty((Bn, s_q, w.h_q), dtype=torch.float32, device="cuda")
    B.gqla_combine_up_proj(bd, op_in.cuda(), lp_in.cuda(), dev["w_uv"], o_f, lse_f)
    errs["combine_up_proj"] = assert_close(o_f.float().cpu().numpy(), O.up_proj(od, oh_ref, f["w_uv"]), "combine_up_proj")
    errs["combine_up_lse"] = assert_close(lse_f.cpu().numpy(), l_ref, "combine_up_proj lse")

    # up_proj on the oracle's o_hat rounded to storage
    oh_in = round_to(w, oh_ref)
    o = torch.empty((Bn, s_q, w.h_q, w.d_h), dtype=dt, device="cuda")
    B.gqla_up_proj(bd, oh_in.cuda(), dev["w_uv"], o)
    errs["up_proj"] = assert_close(o.float().cpu().numpy(), O.up_proj(od, synth.to_f64(oh_in), f["w_uv"]), "up_proj")

    # expand_cache
    N = x["cache"].shape[0]
    k_c = torch.empty((N, w.g, w.d_h), dtype=dt, device="cuda")
    v = torch.empty((N, w.g, w.d_h), dtype=dt, device="cuda")
    k_r = torch.empty((N, w.d_r), dtype=dt, device="cuda")
    B.gqla_expand_cache(bd, dev["cache"], dev["w_uk"], dev["w_uv"], k_c, v, k_r)
    kc_ref, v_ref, kr_ref = O.expand_cache(od, f["cache"], f["w_uk"], f["w_uv"])
    if N > 0:
        errs["expand_k"] = assert_close(k_c.float().cpu().numpy(), kc_ref, "expand k_c")
        errs["expand_v"] = assert_close(v.float().cpu().numpy(), v_ref, "expand v")
        assert np.array_equal(k_r.float().cpu().numpy(), kr_ref), "expand k_r must be a bit-exact copy"

    # decode_gqa on the oracle's expanded cache rounded to storage
    kc_in, v_in, kr_in = round_to(w, kc_ref), round_to(w, v_ref), round_to(w, kr_ref)
    q = torch.cat([x["q_c"], x["q_r"]], dim=-1).contiguous()
    og_part = torch.full((Bn, S, s_q, w.h_q, w.d_h), float("nan"), dtype=torch.float32, device="cuda")
    lg_part = torch.full((Bn, S, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    B.gqla_decode_gqa(bd, q.cuda(), kc_in.cuda(), v_in.cuda(), kr_in.cuda(), dev["seq_start"], dev["seqlens"],
                      w.scale, S, og_part, lg_part, status)
    og_ref, lg_ref = O.decode_gqa_partials(od, synth.to_f64(q), synth.to_f64(kc_in), synth.to_f64(v_in),
                                           synth.to_f64(kr_in), ss, sl, s_q, w.scale, S)
    if check_partials:
        errs["gqa_o_part"] = assert_close(og_part.cpu().numpy(), og_ref, "decode_gqa o_part")
        errs["gqa_lse_part"] = assert_close(lg_part.cpu().numpy(), lg_ref, "decode_gqa lse_part")
    assert int(status.item()) == 0, "device status word set"
    return errs


def end_to_end(w: synth.Workload, seqlens, num_splits: int, q_gain: float = 1.0, sample_seqs=None,
               alias_k_r: bool = True, paths=("absorb", "gqa")):
    """Both full paths through GqlaDecoder from the raw inputs, against the unrounded fp64
    chain.  With sample_seqs the oracle runs only those sequences (all heads, all queries)."""
    od, bd = dims_of(w)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=q_gain)
    dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].cuda(), x["w_uv"].cuda(), x["cache"].cuda(),
                      x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale)
    idx = list(range(w.batch)) if sample_seqs is None else list(sample_seqs)
    ss, sl = x["seq_start"].numpy()[idx], x["seqlens"].numpy()[idx]
    fq_c, fq_r = synth.to_f64(x["q_c"][idx]), synth.to_f64(x["q_r"][idx])
    fw_uk, fw_uv = synth.to_f64(x["w_uk"]), synth.to_f64(x["w_uv"])
    errs = {}
    # the oracle works sequence by sequence so that only one sequence's rows are widened at a time
    def oracle(fn):
        outs = []
        for n, b in enumerate(idx):
            s0, T = int(ss[n]), int(sl[n])
            rows = synth.to_f64(x["cache"][s0:s0 + T])
            outs.append(fn(od, fq_c[n:n + 1], fq_r[n:n + 1], fw_uk, fw_uv, rows, np.zeros(1, dtype=np.int64),
                           np.array([T], dtype=np.int32), w.s_q, w.scale))
        return np.concatenate(outs, axis=0)

    if "absorb" in paths:
        o = dec.absorb_step(x["q_c"].cuda(), x["q_r"].cuda(), num_splits)
        errs["absorb_path"] = assert_close(o.float().cpu().numpy()[idx], oracle(O.absorb_path), "absorb path")
    if "gqa" in paths:
        dec.expand_cache(alias_k_r=alias_k_r)
        q = torch.cat([x["q_c"], x["q_r"]], dim=-1).contiguous().cuda()
        o = dec.gqa_step(q, num_splits)
        errs["gqa_path"] = assert_close(o.float().cpu().numpy()[idx], oracle(O.gqa_path), "gqa path")
    dec.check_status()
    return errs
