"""GPU parity: every C-ABI call against the fp64 oracle on the same seeded inputs.

Bar: bit-exact integer bookkeeping (checked on the host), and for floating point
max|err| <= 1e-2 * max|ref| + 1e-3 (bf16 inputs, fp32 accumulation)."""
import numpy as np
import pytest
import torch

from paper_2605_15250_b200 import binding as B
from paper_2605_15250_b200 import build as gbuild
from paper_2605_15250_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    gbuild.build()
    assert torch.cuda.is_available()
    B.lib()
    yield
    B.set_policy(B.POLICY_AUTO)


@pytest.fixture(params=["auto", "generic"])
def policy(request):
    B.set_policy(B.POLICY_AUTO if request.param == "auto" else B.POLICY_GENERIC)
    yield request.param
    B.set_policy(B.POLICY_AUTO)


CANON = dict(h_q=128, g=8, d_h=128, r_kv=512, d_r=64)
LLAMA = dict(h_q=32, g=8, d_h=128, r_kv=512, d_r=64)


def _wl(name, batch, s_q, seed, dtype="bf16", **dims):
    return synth.Workload(name, batch=batch, s_q=s_q, dtype=dtype, seed=seed, **dims)


def test_c0_tiny_fp32(policy):
    """Workload C0 (tiny check): B=1, h_q=8, g=2, d_h=16, r_kv=32, d_r=8, T=64, fp32."""
    from tests.parity_util import end_to_end, stagewise
    w = synth.WORKLOADS["C0"]
    errs = stagewise(w, None, 1)
    errs.update(end_to_end(w, None, 1))
    # fp32 storage: far inside the bf16 tolerance
    assert max(errs.values()) < 1e-4
    errs = stagewise(w.with_(dtype="bf16"), None, 2)


@pytest.mark.parametrize("s_q", [1, 2, 3])
@pytest.mark.parametrize("S", [1, 3])
def test_odd_shapes_generic(s_q, S):
    """Shapes no specialised kernel covers (h_q/g = 1 and 3, odd dims): generic kernels."""
    from tests.parity_util import end_to_end, stagewise
    B.set_policy(B.POLICY_AUTO)
    w = _wl("odd", 5, s_q, 77, dtype="f32", h_q=6, g=2, d_h=20, r_kv=36, d_r=12)
    seqlens = np.array([0, 1, 2, 65, 200], dtype=np.int32)
    stagewise(w, seqlens, S)
    end_to_end(w, seqlens, S)
    w = _wl("odd2", 3, s_q, 78, dtype="bf16", h_q=4, g=4, d_h=24, r_kv=40, d_r=8)
    stagewise(w, np.array([130, 64, 63], dtype=np.int32), S)


@pytest.mark.parametrize("s_q", [1, 2])
@pytest.mark.parametrize("S,q_gain", [(1, 1.0), (4, 4.0), (9, 4.0)])
def test_canonical_dims_ragged_stagewise(policy, s_q, S, q_gain):
    """Canonical dims, several tiles and ragged tails, empty sequences and T < s_q."""
    from tests.parity_util import stagewise
    w = _wl("canon", 8, s_q, 101, **CANON)
    seqlens = np.array([1, 0, 63, 64, 65, 1000, 129, 2050], dtype=np.int32)
    stagewise(w, seqlens, S, q_gain)


@pytest.mark.parametrize("s_q", [1, 2])
def test_llama_dims_ragged_stagewise(policy, s_q):
    from tests.parity_util import stagewise
    w = _wl("llama", 6, s_q, 102, **LLAMA)
    seqlens = np.array([513, 2, 700, 64, 3000, 127], dtype=np.int32)
    stagewise(w, seqlens, 5, 4.0)


@pytest.mark.parametrize("dims", [CANON, LLAMA])
@pytest.mark.parametrize("s_q,S", [(1, 1), (2, 4)])
def test_end_to_end_mid(policy, dims, s_q, S):
    from tests.parity_util import end_to_end
    w = _wl("mid", 5, s_q, 103, **dims)
    seqlens = np.array([777, 64, 1, 2049, 300], dtype=np.int32)
    end_to_end(w, seqlens, S, q_gain=4.0)
    end_to_end(w, seqlens, S, q_gain=1.0, alias_k_r=False)


def _balanced_gqa_case(w, seqlens, S, q_gain=4.0):
    """GQA path under the balanced plan: every non-empty slot against the oracle's partial on the
    plan the oracle states, unused slots marked -inf, and the merged output against the definition."""
    from oracle import gqla_oracle as O
    from tests.parity_util import assert_close, dims_of
    od, bd = dims_of(w)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=q_gain)
    f = {k: synth.to_f64(v) for k, v in x.items() if k not in ("seq_start", "seqlens")}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    W = B.gqla_balanced_workers(bd, torch.bfloat16, w.s_q, "gqa")
    assert W == torch.cuda.get_device_properties(0).multi_processor_count // w.g
    plans = O.balanced_plan([int(t) for t in sl], S, W)
    assert plans == B.gqla_balanced_plan([int(t) for t in sl], S, W)[0]
    cache = x["cache"].cuda()
    N = cache.shape[0]
    k_c = torch.empty((N, w.g, w.d_h), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(k_c)
    B.gqla_expand_cache(bd, cache, x["w_uk"].cuda(), x["w_uv"].cuda(), k_c, v, None)
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous()
    o_part = torch.full((w.batch, S, w.s_q, w.h_q, w.d_h), float("nan"), dtype=torch.float32, device="cuda")
    lse_part = torch.full((w.batch, S, w.s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gqla_decode_gqa(bd, q.cuda(), k_c, v, cache[:, w.r_kv:], x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale, -S,
                      o_part, lse_part, status)
    out = torch.empty((w.batch, w.s_q, w.h_q, w.d_h), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.batch, w.s_q, w.h_q), dtype=torch.float32, device="cuda")
    B.gqla_combine_splits(o_part, lse_part, out, lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the oracle on the library's own (bf16) expanded cache, so that only the attention is compared
    kc64, v64 = synth.to_f64(k_c), synth.to_f64(v)
    op_ref, lp_ref = O.decode_gqa_partials(od, synth.to_f64(q), kc64, v64, f["cache"][:, w.r_kv:], ss, sl, w.s_q, w.scale,
                                           S, plans)
    got_o, got_l = o_part.cpu().numpy(), lse_part.cpu().numpy()
    live = np.array([[hi > lo for lo, hi in plan] for plan in plans])
    assert np.isneginf(got_l[~live]).all(), "unused slots must carry lse = -inf"
    assert_close(got_l, lp_ref, "balanced lse_part")
    assert_close(got_o[live], op_ref[live], "balanced o_part")
    o_ref, l_ref = O.combine_splits(op_ref, lp_ref)
    assert_close(out.float().cpu().numpy(), o_ref, "balanced merged output")
    assert_close(lse.cpu().numpy(), l_ref, "balanced merged lse")


@pytest.mark.parametrize("s_q", [1, 2])
@pytest.mark.parametrize("S", [2, 5])
def test_gqa_balanced_plan_canonical(s_q, S):
    w = _wl("bal", 9, s_q, 111, **CANON)
    _balanced_gqa_case(w, np.array([1, 0, 63, 2050, 65, 1000, 0, 129, 5000], dtype=np.int32), S)


@pytest.mark.parametrize("s_q", [1, 2])
def test_gqa_balanced_plan_llama_more_workers_than_tiles(s_q):
    w = _wl("bal2", 3, s_q, 112, **LLAMA)
    _balanced_gqa_case(w, np.array([130, 0, 300], dtype=np.int32), 2)
    w = _wl("bal3", 40, s_q, 113, **LLAMA)
    _balanced_gqa_case(w, synth.make_seqlens(w.with_(seqlen_range=(0, 1500))), 3)


def _balanced_absorb_case(w, seqlens, S, q_gain=4.0):
    """Absorb path under the balanced plan: same checks as _balanced_gqa_case."""
    from oracle import gqla_oracle as O
    from tests.parity_util import assert_close, dims_of
    od, bd = dims_of(w)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=q_gain)
    f = {k: synth.to_f64(v) for k, v in x.items() if k not in ("seq_start", "seqlens")}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    W = B.gqla_balanced_workers(bd, torch.bfloat16, w.s_q, "absorb")
    assert W >= 1
    plans = O.balanced_plan([int(t) for t in sl], S, W)
    q_hat = torch.from_numpy(O.absorb_q(od, f["q_c"], f["q_r"], f["w_uk"])).to(torch.bfloat16)
    o_part = torch.full((w.batch, S, w.s_q, w.h_q, w.r_kv), float("nan"), dtype=torch.float32, device="cuda")
    lse_part = torch.full((w.batch, S, w.s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.gqla_decode_absorb(bd, q_hat.cuda(), x["cache"].cuda(), x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale, -S,
                         o_part, lse_part, status)
    out = torch.empty((w.batch, w.s_q, w.h_q, w.r_kv), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.batch, w.s_q, w.h_q), dtype=torch.float32, device="cuda")
    B.gqla_combine_splits(o_part, lse_part, out, lse)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    op_ref, lp_ref = O.decode_absorb_partials(od, synth.to_f64(q_hat), f["cache"], ss, sl, w.s_q, w.scale, S, plans)
    got_o, got_l = o_part.cpu().numpy(), lse_part.cpu().numpy()
    live = np.array([[hi > lo for lo, hi in plan] for plan in plans])
    assert np.isneginf(got_l[~live]).all(), "unused slots must carry lse = -inf"
    assert_close(got_l, lp_ref, "balanced lse_part")
    assert_close(got_o[live], op_ref[live], "balanced o_part")
    o_ref, l_ref = O.combine_splits(op_ref, lp_ref)
    assert_close(out.float().cpu().numpy(), o_ref, "balanced merged output")
    assert_close(lse.cpu().numpy(), l_ref, "balanced merged lse")


@pytest.mark.parametrize("s_q", [1, 2])
@pytest.mark.parametrize("S", [2, 5])
def test_absorb_balanced_plan_canonical(s_q, S):
    w = _wl("abal", 9, s_q, 121, **CANON)
    _balanced_absorb_case(w, np.array([1, 0, 63, 2050, 65, 1000, 0, 129, 5000], dtype=np.int32), S)


@pytest.mark.parametrize("s_q", [1, 2])
def test_absorb_balanced_plan_llama(s_q):
    w = _wl("abal2", 3, s_q, 122, **LLAMA)
    _balanced_absorb_case(w, np.array([130, 0, 300], dtype=np.int32), 2)
    w = _wl("abal3", 200, s_q, 123, **LLAMA)
    _balanced_absorb_case(w, synth.make_seqlens(w.with_(seqlen_range=(0, 1500))), 3)


@pytest.mark.parametrize("h_q,g", [(128, 4), (64, 8), (64, 4), (16, 8), (28, 4), (20, 4)])
@pytest.mark.parametrize("s_q", [1, 2])
def test_shape_variants_of_the_paper(h_q, g, s_q):
    """Operating points the paper discusses besides the canonical one: g = 4 (cache 2176 B/token, Table
    "roofline"), h_q = 64 (Sec. 4.2), few heads per group, and head counts whose heads per group are not a
    power of two (h_q = 28 at g = 4, the Qwen2.5-7B setup of Sec. 5; h_q = 20); fixed and balanced plans.
    Both decode paths stay on the tensor-core kernels."""
    from tests.parity_util import end_to_end, stagewise
    dims = B.make_dims(h_q, g, 128, 512, 64)
    assert B.kernel_for(dims, torch.bfloat16, s_q, "absorb") == "tcgen05"
    assert B.kernel_for(dims, torch.bfloat16, s_q, "gqa") == "tcgen05"
    assert B.kernel_for(dims, torch.bfloat16, s_q, "projections") == "tcgen05"
    w = _wl("variant", 5, s_q, 131, h_q=h_q, g=g, d_h=128, r_kv=512, d_r=64)
    seqlens = np.array([700, 0, 129, 2050, 64], dtype=np.int32)
    stagewise(w, seqlens, 3, 4.0)
    end_to_end(w, seqlens, -3, q_gain=4.0)


@pytest.mark.parametrize("dims", [CANON, LLAMA])
@pytest.mark.parametrize("s_q", [1, 2])
@pytest.mark.parametrize("page_size,S", [(128, 1), (128, -3), (256, -3), (128, 3), (16, 2), (48, -3)])
def test_paged_cache_gives_what_the_packed_cache_gives(dims, s_q, page_size, S):
    """Paging is storage only (the paper's model leaves it out, Sec. 5.1): both decode calls over a pool of
    shuffled pages must return what they return over the packed cache that holds the same rows -- bit for
    bit where both runs use the same kernel and the same pieces (tensor-core kernels: pages of a multiple
    of 128 rows with one split or the balanced plan; generic kernels: any page size) -- and match the oracle
    fed with the rows gathered back."""
    from tests.parity_util import assert_close, dims_of, round_to
    from oracle import gqla_oracle as O
    w = _wl("paged", 5, s_q, 160, **dims)
    seqlens = np.array([700, 0, 129, 2050, 1], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=4.0)
    od, bd = dims_of(w)
    slots = abs(S)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    sl = x["seqlens"].cuda()
    cache_p, table = synth.to_paged(x["cache"], x["seq_start"], seqlens, page_size, seed=161)
    table_d = table.cuda()
    f = {k: synth.to_f64(x[k]) for k in ("q_c", "q_r", "cache", "w_uk", "w_uv")}
    # the oracle reads the pool through its own gather
    rows, ss = O.unpage(synth.to_f64(cache_p), table.numpy(), page_size, seqlens)
    assert np.array_equal(rows, f["cache"])

    # ---- absorb path
    qh_in = round_to(w, O.absorb_q(od, f["q_c"], f["q_r"], f["w_uk"])).cuda()

    def parts(D):
        return (torch.full((w.batch, slots, s_q, w.h_q, D), float("nan"), dtype=torch.float32, device="cuda"),
                torch.full((w.batch, slots, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda"))

    o_a, l_a = parts(w.r_kv)
    B.gqla_decode_absorb(bd, qh_in, x["cache"].cuda(), x["seq_start"].cuda(), sl, w.scale, S, o_a, l_a, status)
    o_b, l_b = parts(w.r_kv)
    B.gqla_decode_absorb_paged(bd, qh_in, cache_p.cuda(), table_d, page_size, sl, w.scale, S, o_b, l_b, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    same_kernel = page_size % 128 == 0 and (S == 1 or S < 0)  # else the paged call runs on the generic kernel
    live = ~torch.isneginf(l_a)  # partial outputs of empty slots are not written under the balanced plan
    if same_kernel:  # same pieces too; otherwise only the merged result is comparable (below)
        assert torch.equal(l_a, l_b) and torch.equal(o_a[live], o_b[live])
    oh = torch.empty((w.batch, s_q, w.h_q, w.r_kv), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.batch, s_q, w.h_q), dtype=torch.float32, device="cuda")
    B.gqla_combine_splits(o_b, l_b, oh, lse)
    oh_ref, lse_ref = O.decode_absorb(od, synth.to_f64(qh_in), rows, ss, seqlens, s_q, w.scale)
    assert_close(oh.float().cpu().numpy(), oh_ref, "paged absorb o_hat")
    assert_close(lse.cpu().numpy(), lse_ref, "paged absorb lse")

    # ---- GQA path: the expansion is per row, so the pool is expanded as it is
    N_p = cache_p.shape[0]
    kc_p = torch.empty((N_p, w.g, w.d_h), dtype=torch.bfloat16, device="cuda")
    v_p = torch.empty_like(kc_p)
    cache_pd = cache_p.cuda()
    B.gqla_expand_cache(bd, cache_pd, x["w_uk"].cuda(), x["w_uv"].cuda(), kc_p, v_p, None)
    N = x["cache"].shape[0]
    kc = torch.empty((N, w.g, w.d_h), dtype=torch.bfloat16, device="cuda")
    v = torch.empty_like(kc)
    cache_d = x["cache"].cuda()
    B.gqla_expand_cache(bd, cache_d, x["w_uk"].cuda(), x["w_uv"].cuda(), kc, v, None)
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
    o_a, l_a = parts(w.d_h)
    B.gqla_decode_gqa(bd, q, kc, v, cache_d[:, w.r_kv:], x["seq_start"].cuda(), sl, w.scale, S, o_a, l_a, status)
    o_b, l_b = parts(w.d_h)
    B.gqla_decode_gqa_paged(bd, q, kc_p, v_p, cache_pd[:, w.r_kv:], table_d, page_size, sl, w.scale, S, o_b, l_b, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    live = ~torch.isneginf(l_a)
    if same_kernel:  # same pieces too; otherwise only the merged result is comparable (below)
        assert torch.equal(l_a, l_b) and torch.equal(o_a[live], o_b[live])
    o = torch.empty((w.batch, s_q, w.h_q, w.d_h), dtype=torch.bfloat16, device="cuda")
    B.gqla_combine_splits(o_b, l_b, o, None)
    o_ref = O.gqa_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], rows, ss, seqlens, s_q, w.scale)
    assert_close(o.float().cpu().numpy(), o_ref, "paged gqa path")


def test_decoder_chains_over_a_paged_cache():
    """GqlaDecoder with a block table: both chains (absorb with the fused tail, GQA after expanding the
    whole pool) against the oracle on the rows gathered back."""
    from tests.parity_util import assert_close, dims_of
    from oracle import gqla_oracle as O
    from paper_2605_15250_b200.decoder import GqlaDecoder
    s_q, page_size = 2, 128
    w = _wl("pagedec", 4, s_q, 170, **CANON)
    seqlens = np.array([900, 3, 0, 260], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=4.0)
    od, _ = dims_of(w)
    cache_p, table = synth.to_paged(x["cache"], x["seq_start"], seqlens, page_size, seed=171)
    dev = torch.device("cuda", 0)
    dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].to(dev), x["w_uv"].to(dev), cache_p.to(dev), None,
                      x["seqlens"].to(dev), w.scale, block_table=table.to(dev), page_size=page_size)
    f = {k: synth.to_f64(x[k]) for k in ("q_c", "q_r", "w_uk", "w_uv")}
    rows, ss = O.unpage(synth.to_f64(cache_p), table.numpy(), page_size, seqlens)
    o = dec.absorb_step(x["q_c"].to(dev), x["q_r"].to(dev), -3)
    assert_close(o.float().cpu().numpy(), O.absorb_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], rows, ss, seqlens, s_q,
                                                        w.scale), "paged absorb chain")
    dec.expand_cache()
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().to(dev)
    o = dec.gqa_step(q, -2)
    dec.check_status()
    assert_close(o.float().cpu().numpy(), O.gqa_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], rows, ss, seqlens, s_q,
                                                     w.scale), "paged gqa chain")
    with pytest.raises(B.GqlaError):
        dec.append_expand(s_q)


@pytest.mark.parametrize("hpg,g,s_q", [(1, 8, 1), (1, 4, 8), (3, 2, 1), (3, 4, 5), (5, 4, 3), (6, 2, 2), (7, 4, 4), (9, 1, 6),
                                       (12, 2, 7), (24, 4, 2), (32, 2, 3), (64, 1, 2), (128, 1, 1)])
def test_heads_per_group_and_query_counts_off_the_powers_of_two(hpg, g, s_q):
    """Heads per group and query positions are padded to powers of two inside the tensor-core kernels
    (padding rows read zeros or a neighbour's queries and are dropped at the store).  Every combination
    here has padding on one or both axes, or sits at an edge (one head per group, 128 rows per group);
    both paths, fixed and balanced plans, against the oracle."""
    from tests.parity_util import end_to_end
    dims = B.make_dims(hpg * g, g, 128, 512, 64)
    for path in ("absorb", "gqa", "projections"):
        assert B.kernel_for(dims, torch.bfloat16, s_q, path) == "tcgen05", path
    w = _wl("pad", 4, s_q, 150 + hpg + s_q, h_q=hpg * g, g=g, d_h=128, r_kv=512, d_r=64)
    seqlens = np.array([300, max(s_q - 1, 0), 129, 517], dtype=np.int32)
    end_to_end(w, seqlens, 2, q_gain=4.0)
    end_to_end(w, seqlens, -3, q_gain=4.0)


@pytest.mark.parametrize("dims,dtype", [(CANON, "bf16"), (LLAMA, "bf16"),
                                        (dict(h_q=6, g=2, d_h=20, r_kv=36, d_r=12), "f32")])
@pytest.mark.parametrize("s_q", [1, 2, 3])
@pytest.mark.parametrize("copy_k_r", [False, True])
def test_append_expand_touches_only_the_new_rows(dims, dtype, s_q, copy_k_r):
    """The expansion of Sec. 3.1 is a per-token map: after a step only the s_q rows each sequence appended
    need expanding.  The new rows must equal the oracle's expansion of those rows, k_R bit for bit, and every
    other row of the planes must keep the sentinel it held (also for sequences shorter than s_q)."""
    from tests.parity_util import assert_close, dims_of
    from oracle import gqla_oracle as O
    w = _wl("append", 7, s_q, 140, dtype=dtype, **dims)
    seqlens = np.array([700, 0, 1, 129, 2050, 2, 64], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens)
    od, bd = dims_of(w)
    dt = x["cache"].dtype
    N = x["cache"].shape[0]
    sentinel = 7.0
    k_c = torch.full((N, w.g, w.d_h), sentinel, dtype=dt, device="cuda")
    v = torch.full((N, w.g, w.d_h), sentinel, dtype=dt, device="cuda")
    k_r = torch.full((N, w.d_r), sentinel, dtype=dt, device="cuda") if copy_k_r else None
    B.gqla_append_expand(bd, s_q, x["cache"].cuda(), x["seq_start"].cuda(), x["seqlens"].cuda(), x["w_uk"].cuda(),
                         x["w_uv"].cuda(), k_c, v, k_r)
    torch.cuda.synchronize()
    f = {k: synth.to_f64(x[k]) for k in ("cache", "w_uk", "w_uv")}
    kc_ref, v_ref, kr_ref = O.expand_cache(od, f["cache"], f["w_uk"], f["w_uv"])
    new = np.zeros(N, dtype=bool)
    for b, T in enumerate(seqlens):
        for pos in range(max(0, int(T) - s_q), int(T)):
            new[int(x["seq_start"][b]) + pos] = True
    assert new.sum() == sum(min(int(T), s_q) for T in seqlens)
    kc_got, v_got = k_c.float().cpu().numpy(), v.float().cpu().numpy()
    assert_close(kc_got[new], kc_ref[new], "append k_c")
    assert_close(v_got[new], v_ref[new], "append v")
    assert np.all(kc_got[~new] == sentinel) and np.all(v_got[~new] == sentinel), "rows outside the step were written"
    if copy_k_r:
        kr_got = k_r.float().cpu().numpy()
        assert np.array_equal(kr_got[new], kr_ref[new]), "k_R of the new rows must be a bit-exact copy"
        assert np.all(kr_got[~new] == sentinel)


def test_append_expand_keeps_an_expanded_cache_current():
    """A decode loop on the GQA path: expand once, then per step append s_q latent rows per sequence and
    expand only those.  Attention over the incrementally kept planes must agree with the oracle's GQA path
    on the grown cache."""
    from tests.parity_util import assert_close, dims_of
    from oracle import gqla_oracle as O
    from paper_2605_15250_b200.decoder import GqlaDecoder
    s_q = 2
    w = _wl("loop", 3, s_q, 141, **CANON)
    final = np.array([260, 131, 7], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=final, q_gain=4.0)
    od, bd = dims_of(w)
    dev = torch.device("cuda", 0)
    steps = 3
    # the cache starts steps * s_q rows short; each step reveals s_q more rows per sequence
    start = np.maximum(final - steps * s_q, 0).astype(np.int32)
    dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].to(dev), x["w_uv"].to(dev), x["cache"].to(dev),
                      x["seq_start"].to(dev), torch.from_numpy(start).to(dev), w.scale)
    dec.expand_cache()
    # rows beyond the start lengths are wiped, so that stale values cannot pass for appended ones
    keep = np.zeros(x["cache"].shape[0], dtype=bool)
    for b, T in enumerate(start):
        keep[int(x["seq_start"][b]):int(x["seq_start"][b]) + int(T)] = True
    wipe = torch.from_numpy(~keep).to(dev)
    dec.k_c[wipe] = 0
    dec.v[wipe] = 0
    cur = start.copy()
    for _ in range(steps):
        cur = np.minimum(cur + s_q, final).astype(np.int32)
        dec.seqlens.copy_(torch.from_numpy(cur))
        dec.append_expand(s_q)
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().to(dev)
    o = dec.gqa_step(q, 2)
    torch.cuda.synchronize()
    dec.check_status()
    f = {k: synth.to_f64(x[k]) for k in ("q_c", "q_r", "cache", "w_uk", "w_uv")}
    o_ref = O.gqa_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], x["seq_start"].numpy(), final, s_q,
                       w.scale)
    assert_close(o.float().cpu().numpy(), o_ref, "gqa path after incremental expansion")


@pytest.mark.parametrize("s_q", [3, 4, 5, 8])
def test_speculative_query_counts(s_q):
    """s_q >= 3 (speculative decoding, Sec. 4.2): both paths stay on the tensor-core kernels (the absorb
    path with more row blocks, the GQA path with s_q = 3 padded to four query positions per head); the
    causal mask covers all s_q positions."""
    from tests.parity_util import end_to_end, stagewise
    w = _wl("spec", 4, s_q, 132, **CANON)
    assert B.kernel_for(B.make_dims(**CANON), torch.bfloat16, s_q, "absorb") == "tcgen05"
    assert B.kernel_for(B.make_dims(**CANON), torch.bfloat16, s_q, "gqa") == "tcgen05"
    seqlens = np.array([300, 2, 1029, 64], dtype=np.int32)
    stagewise(w, seqlens, 2, 4.0)
    end_to_end(w, seqlens, 2, q_gain=4.0)
    end_to_end(w, seqlens, -3, q_gain=4.0)


def test_two_gpu_paths_agree_with_each_other():
    """Same weights, same latent: the two paths' GPU outputs differ by at most twice the
    tolerance (each is within it of the same oracle value)."""
    from tests.parity_util import ABS, REL
    from paper_2605_15250_b200.decoder import GqlaDecoder
    w = _wl("agree", 4, 2, 104, **CANON)
    x = synth.make_inputs(w, seqlens=np.array([500, 1200, 64, 333], dtype=np.int32), q_gain=4.0)
    dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].cuda(), x["w_uv"].cuda(), x["cache"].cuda(),
                      x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale)
    a = dec.absorb_step(x["q_c"].cuda(), x["q_r"].cuda(), 2).float().cpu()
    dec.expand_cache()
    gq = dec.gqa_step(torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda(), 2).float().cpu()
    assert (a - gq).abs().max().item() <= 2 * (REL * a.abs().max().item() + ABS)


def test_random_batches_fixed_and_balanced_plans_agree():
    """Many small random batches (empty and one-row sequences included) through both kernels under
    both plans: the merged outputs of the two plans must agree (they are partitions of the same sum),
    the status word must stay clear, and repeated launches must not interfere (persistent CTAs keep
    barrier phases across pieces)."""
    from tests.parity_util import ABS, REL
    from paper_2605_15250_b200.decoder import GqlaDecoder
    rng = np.random.default_rng(2024)
    for it in range(40):
        dims = CANON if it % 2 == 0 else LLAMA
        s_q = 1 + it % 2 if it % 4 < 2 else 2 - it % 2
        nb = int(rng.integers(1, 24))
        sl = rng.integers(0, 3000, size=nb).astype(np.int32)
        sl[rng.integers(0, nb, size=max(1, nb // 5))] = rng.integers(0, 3, size=max(1, nb // 5))
        w = _wl("rand", nb, s_q, 900 + it, **dims)
        x = synth.make_inputs(w, seqlens=sl, q_gain=3.0)
        dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].cuda(), x["w_uv"].cuda(), x["cache"].cuda(),
                          x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale)
        qc, qr = x["q_c"].cuda(), x["q_r"].cuda()
        q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
        dec.expand_cache()
        S_fixed, S_bal = int(rng.integers(1, 6)), -int(rng.integers(2, 6))
        a_f = dec.absorb_step(qc, qr, S_fixed).float().clone()
        a_b = dec.absorb_step(qc, qr, S_bal).float().clone()
        g_f = dec.gqa_step(q, S_fixed).float().clone()
        g_b = dec.gqa_step(q, S_bal).float().clone()
        dec.check_status()
        for name, u, v in (("absorb", a_f, a_b), ("gqa", g_f, g_b), ("paths", a_b, g_b)):
            assert not torch.isnan(u).any() and not torch.isnan(v).any(), (it, name)
            bound = (2 if name == "paths" else 1) * (REL * u.abs().max().item() + ABS)
            assert (u - v).abs().max().item() <= bound, (it, name, sl.tolist(), S_fixed, S_bal)


def test_determinism_run_to_run():
    from paper_2605_15250_b200.decoder import GqlaDecoder
    w = _wl("det", 4, 2, 105, **CANON)
    x = synth.make_inputs(w, seqlens=np.array([900, 4000, 65, 2048], dtype=np.int32))
    dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].cuda(), x["w_uv"].cuda(), x["cache"].cuda(),
                      x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale)
    qc, qr = x["q_c"].cuda(), x["q_r"].cuda()
    a1 = dec.absorb_step(qc, qr, 4).clone()
    a2 = dec.absorb_step(qc, qr, 4).clone()
    assert torch.equal(a1, a2)
    # the GQA kernel, and both kernels under the balanced plan (no global counters: the cut points are a pure
    # function of the lengths, so the reduction order is fixed there too)
    dec.expand_cache()
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
    for S in (4, 1, -3):
        g1 = dec.gqa_step(q, S).clone()
        g2 = dec.gqa_step(q, S).clone()
        assert torch.equal(g1, g2), S
    b1 = dec.absorb_step(qc, qr, -3).clone()
    b2 = dec.absorb_step(qc, qr, -3).clone()
    assert torch.equal(b1, b2)
    f1 = dec.absorb_step(qc, qr, 1).clone()
    f2 = dec.absorb_step(qc, qr, 1).clone()
    assert torch.equal(f1, f2)
    dec.check_status()


# ------------------------------------------------------------------ overruns and index checks


def test_outputs_do_not_overrun_their_buffers():
    """Every output of the tensor-core kernels sits between guard regions: bulk and TMA stores clipped at ragged
    ends (N not a multiple of the 128 / 256-row tiles, h_q not a multiple of the row block), partial slots, final rows."""
    from tests.parity_util import Canaried
    w = _wl("canary", 3, 2, 211, **dict(h_q=28, g=4, d_h=128, r_kv=512, d_r=64))
    seqlens = np.array([333, 1, 1291], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens)
    bd = B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    dev = {k: t.cuda() for k, t in x.items()}
    N, Bn, s_q = x["cache"].shape[0], w.batch, w.s_q
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bf, f32 = torch.bfloat16, torch.float32
    q_hat = Canaried((Bn, s_q, w.h_q, w.d_abs), bf)
    B.gqla_absorb_q(bd, dev["q_c"], dev["q_r"], dev["w_uk"], q_hat.t)
    k_c, v, k_r = Canaried((N, w.g, w.d_h), bf), Canaried((N, w.g, w.d_h), bf), Canaried((N, w.d_r), bf)
    B.gqla_expand_cache(bd, dev["cache"], dev["w_uk"], dev["w_uv"], k_c.t, v.t, k_r.t)
    outs = [(q_hat, "absorb_q"), (k_c, "expand k_c"), (v, "expand v"), (k_r, "expand k_r")]
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
    for S in (1, 3, -3):
        sl = abs(S)
        oa, la = Canaried((Bn, sl, s_q, w.h_q, w.r_kv), f32), Canaried((Bn, sl, s_q, w.h_q), f32)
        B.gqla_decode_absorb(bd, q_hat.t, dev["cache"], dev["seq_start"], dev["seqlens"], w.scale, S, oa.t, la.t, status)
        og, lg = Canaried((Bn, sl, s_q, w.h_q, w.d_h), f32), Canaried((Bn, sl, s_q, w.h_q), f32)
        B.gqla_decode_gqa(bd, q, k_c.t, v.t, k_r.t, dev["seq_start"], dev["seqlens"], w.scale, S, og.t, lg.t, status)
        o_f, l_f = Canaried((Bn, s_q, w.h_q, w.d_h), bf), Canaried((Bn, s_q, w.h_q), f32)
        B.gqla_combine_up_proj(bd, oa.t, la.t, dev["w_uv"], o_f.t, l_f.t)
        o_c = Canaried((Bn, s_q, w.h_q, w.d_h), bf)
        B.gqla_combine_splits(og.t, lg.t, o_c.t, None)
        outs += [(oa, f"absorb o_part S={S}"), (la, f"absorb lse_part S={S}"), (og, f"gqa o_part S={S}"), (lg, f"gqa lse_part S={S}"),
                 (o_f, f"combine_up_proj S={S}"), (l_f, f"combine_up_proj lse S={S}"), (o_c, f"combine_splits S={S}")]
    o_hat, lse = Canaried((Bn, s_q, w.h_q, w.r_kv), bf), Canaried((Bn, s_q, w.h_q), f32)
    B.gqla_decode_absorb_final(bd, q_hat.t, dev["cache"], dev["seq_start"], dev["seqlens"], w.scale, o_hat.t, lse.t, status)
    o = Canaried((Bn, s_q, w.h_q, w.d_h), bf)
    B.gqla_up_proj(bd, o_hat.t, dev["w_uv"], o.t)
    B.gqla_append_expand(bd, s_q, dev["cache"], dev["seq_start"], dev["seqlens"], dev["w_uk"], dev["w_uv"], k_c.t, v.t, k_r.t)
    outs += [(o_hat, "decode_absorb_final"), (lse, "decode_absorb_final lse"), (o, "up_proj"), (k_c, "append k_c"), (v, "append v"),
             (k_r, "append k_r")]
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for c, what in outs:
        c.check(what)


@pytest.mark.parametrize("kernel", ["rows", "tokens"])
def test_both_gqa_kernels_on_the_shapes_both_cover(kernel):
    """Two tensor-core kernels serve the GQA path: tokens on the MMA's M axis (few query rows per group; the default
    up to 32 padded rows) and replicated query rows.  GQLA_GQA_KERNEL forces either one where both apply; the choice
    is read once per process, so each runs the ragged parity cases in a process of its own."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import numpy as np, torch\n"
        "from paper_2605_15250_b200 import binding as B, synth\n"
        "from tests.parity_util import end_to_end, stagewise\n"
        "sl = np.array([700, 0, 129, 2050, 64, 1], dtype=np.int32)\n"
        "for dims, s_q in ((dict(h_q=128, g=8, d_h=128, r_kv=512, d_r=64), 2), (dict(h_q=128, g=8, d_h=128, r_kv=512, d_r=64), 1),\n"
        "                  (dict(h_q=32, g=8, d_h=128, r_kv=512, d_r=64), 2), (dict(h_q=28, g=4, d_h=128, r_kv=512, d_r=64), 3),\n"
        "                  (dict(h_q=128, g=8, d_h=128, r_kv=512, d_r=64), 4)):\n"
        "    w = synth.Workload('k', batch=6, s_q=s_q, dtype='bf16', seed=9, **dims)\n"
        "    stagewise(w, sl, 3, q_gain=4.0)\n"
        "    for S in (1, -3):\n"
        "        end_to_end(w, sl, S, q_gain=4.0, paths=('gqa',))\n"
        "print('kernel-ok')\n")
    env = dict(os.environ, GQLA_GQA_KERNEL=kernel, PYTHONPATH=root)
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, cwd=root, timeout=900)
    assert res.returncode == 0 and "kernel-ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


@pytest.mark.parametrize("kernel", ["rows", "tokens"])
def test_both_absorb_kernels_on_the_shapes_both_cover(kernel):
    """Two tensor-core kernels serve the absorb path: tokens on the MMA's M axis for h_q * s_q <= 64 (every cache tile
    fetched once and used as K and as V) and the CTA-pair kernel with the query rows on M.
    GQLA_ABSORB_KERNEL forces either one where both apply; the choice is read once per process, so each runs the
    ragged parity cases (fixed, balanced and whole-sequence plans) in a process of its own."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import numpy as np, torch\n"
        "from paper_2605_15250_b200 import binding as B, synth\n"
        "from tests.parity_util import end_to_end, stagewise\n"
        "sl = np.array([700, 0, 129, 2050, 64, 1, 63, 65], dtype=np.int32)\n"
        "for dims, s_q in ((dict(h_q=32, g=8, d_h=128, r_kv=512, d_r=64), 1), (dict(h_q=16, g=8, d_h=128, r_kv=512, d_r=64), 2),\n"
        "                  (dict(h_q=28, g=4, d_h=128, r_kv=512, d_r=64), 1), (dict(h_q=8, g=8, d_h=128, r_kv=512, d_r=64), 2),\n"
        "                  (dict(h_q=8, g=4, d_h=128, r_kv=512, d_r=64), 3), (dict(h_q=32, g=8, d_h=128, r_kv=512, d_r=64), 2),\n"
        "                  (dict(h_q=20, g=4, d_h=128, r_kv=512, d_r=64), 3)):\n"
        "    w = synth.Workload('k', batch=8, s_q=s_q, dtype='bf16', seed=9, **dims)\n"
        "    d = B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)\n"
        "    sms = torch.cuda.get_device_properties(0).multi_processor_count\n"
        "    assert B.gqla_balanced_workers(d, torch.bfloat16, s_q, 'absorb') == (sms if '%s' == 'tokens' else sms // 2)\n"
        "    stagewise(w, sl, 3, q_gain=4.0)\n"
        "    for S in (1, 4, -3):\n"
        "        end_to_end(w, sl, S, q_gain=4.0, paths=('absorb',))\n"
        "print('kernel-ok')\n") % kernel
    env = dict(os.environ, GQLA_ABSORB_KERNEL=kernel, PYTHONPATH=root)
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, cwd=root, timeout=900)
    assert res.returncode == 0 and "kernel-ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


def test_debug_build_index_checks_stay_silent():
    """The -DGQLA_DEBUG build (piece and tile index checks that record a code instead of trapping) runs the ragged
    parity case in a process of its own: outputs within tolerance, status word 0."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    lib = gbuild.build(debug=True)
    code = (
        "import numpy as np, torch\n"
        "from paper_2605_15250_b200 import binding as B, synth\n"
        "from tests.parity_util import end_to_end\n"
        "assert B.LIB_PATH.endswith('libgqla_debug.so')\n"
        "sl = np.array([700, 0, 129, 2050, 64], dtype=np.int32)\n"
        "for h_q in (128, 32):  # query rows on the MMA's M axis / tokens on M, on both paths\n"
        "    w = synth.Workload('dbg', h_q, 8, 128, 512, 64, batch=5, s_q=2, dtype='bf16', seed=5)\n"
        "    for S in (1, 3, -3):\n"
        "        end_to_end(w, sl, S, q_gain=4.0)\n"
        "print('debug-ok')\n")
    env = dict(os.environ, GQLA_LIB_PATH=lib, PYTHONPATH=root)
    res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, env=env, cwd=root, timeout=600)
    assert res.returncode == 0 and "debug-ok" in res.stdout, res.stdout[-2000:] + res.stderr[-4000:]


# ------------------------------------------------------------------ a value head dimension of its own


@pytest.mark.parametrize("dims,d_v,dtype", [(dict(h_q=20, g=4, d_h=192, r_kv=512, d_r=64), 256, "bf16"),   # GLM-like
                                            (dict(h_q=32, g=8, d_h=128, r_kv=512, d_r=64), 256, "bf16"),
                                            (dict(h_q=8, g=2, d_h=16, r_kv=32, d_r=8), 24, "f32")])
def test_separate_value_head_dim(dims, d_v, dtype):
    """Sec. 3.2 "From MLA to GQLA": d_h^V != d_h.  Both paths through the *_dv calls against the oracle, stage by
    stage where d_v enters (expansion, GQA attention, up-projection) and end to end."""
    from tests.parity_util import assert_close
    from oracle import gqla_oracle as O
    w = synth.Workload("dv", batch=3, s_q=2, dtype=dtype, seed=77, d_v=d_v, **dims)
    seqlens = np.array([300, 1, 1029], dtype=np.int32)
    x = synth.make_inputs(w, seqlens=seqlens, q_gain=3.0)
    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, d_v)
    bd = B.make_dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    td = torch.bfloat16 if dtype == "bf16" else torch.float32
    dev = {k: t.cuda() for k, t in x.items()}
    f = {k: synth.to_f64(t) for k, t in x.items() if k not in ("seq_start", "seqlens")}
    ss, sl = x["seq_start"].numpy(), x["seqlens"].numpy()
    N, Bn, s_q, S = x["cache"].shape[0], w.batch, w.s_q, 3
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # expansion
    k_c = torch.empty((N, w.g, w.d_h), dtype=td, device="cuda")
    v = torch.empty((N, w.g, d_v), dtype=td, device="cuda")
    k_r = torch.empty((N, w.d_r), dtype=td, device="cuda")
    B.gqla_expand_cache_dv(bd, dev["cache"], dev["w_uk"], dev["w_uv"], k_c, v, k_r)
    kc_ref, v_ref, kr_ref = O.expand_cache(od, f["cache"], f["w_uk"], f["w_uv"])
    assert_close(k_c.float().cpu().numpy(), kc_ref, "expand_dv k_c")
    assert_close(v.float().cpu().numpy(), v_ref, "expand_dv v")
    assert np.array_equal(k_r.float().cpu().numpy(), kr_ref)
    # GQA path on the library's own planes, against the oracle on those planes and on the unrounded chain
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous()
    o_part = torch.full((Bn, S, s_q, w.h_q, d_v), float("nan"), dtype=torch.float32, device="cuda")
    lse_part = torch.full((Bn, S, s_q, w.h_q), float("nan"), dtype=torch.float32, device="cuda")
    B.gqla_decode_gqa_dv(bd, q.cuda(), k_c, v, k_r, dev["seq_start"], dev["seqlens"], w.scale, S, o_part, lse_part, status)
    op_ref, lp_ref = O.decode_gqa_partials(od, synth.to_f64(q), synth.to_f64(k_c), synth.to_f64(v), synth.to_f64(k_r), ss, sl,
                                           s_q, w.scale, S)
    assert_close(o_part.cpu().numpy(), op_ref, "decode_gqa_dv o_part")
    assert_close(lse_part.cpu().numpy(), lp_ref, "decode_gqa_dv lse_part")
    o_g = torch.empty((Bn, s_q, w.h_q, d_v), dtype=td, device="cuda")
    B.gqla_combine_splits(o_part, lse_part, o_g, None)
    ref = O.gqa_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], ss, sl, s_q, w.scale)
    assert ref.shape[-1] == d_v
    assert_close(o_g.float().cpu().numpy(), ref, "gqa path with d_v")
    # absorb path: the latent attention is unchanged, the up-projection is d_v wide
    q_hat = torch.empty((Bn, s_q, w.h_q, w.d_abs), dtype=td, device="cuda")
    B.gqla_absorb_q(bd, dev["q_c"], dev["q_r"], dev["w_uk"], q_hat)
    oa_part = torch.empty((Bn, S, s_q, w.h_q, w.r_kv), dtype=torch.float32, device="cuda")
    la_part = torch.empty((Bn, S, s_q, w.h_q), dtype=torch.float32, device="cuda")
    B.gqla_decode_absorb(bd, q_hat, dev["cache"], dev["seq_start"], dev["seqlens"], w.scale, S, oa_part, la_part, status)
    o_hat = torch.empty((Bn, s_q, w.h_q, w.r_kv), dtype=td, device="cuda")
    B.gqla_combine_splits(oa_part, la_part, o_hat, None)
    o_a = torch.empty((Bn, s_q, w.h_q, d_v), dtype=td, device="cuda")
    B.gqla_up_proj_dv(bd, o_hat, dev["w_uv"], o_a)
    assert_close(o_a.float().cpu().numpy(), O.up_proj(od, synth.to_f64(o_hat), f["w_uv"]), "up_proj_dv")
    assert_close(o_a.float().cpu().numpy(), ref, "absorb path with d_v")
    assert int(status.item()) == 0


# ------------------------------------------------------------------ workloads C1-C4 at full size


def test_c1_full_absorb():
    """Config 1: h_q=128, g=8, B=64, T=4096, s_q=1, absorb path (as the benchmark launches it)."""
    from tests.parity_util import end_to_end
    end_to_end(synth.WORKLOADS["C1"], None, 1, paths=("absorb",))
    # the same launch on the peaked inputs (O(1) outputs: the relative term of the bound decides), every sequence
    end_to_end(synth.WORKLOADS["C1"], None, 1, q_gain=4.0, paths=("absorb",))


def test_c2_full_gqa_mtp():
    """Config 2: same weights and latent, expanded cache, s_q=2 causal."""
    from tests.parity_util import end_to_end
    end_to_end(synth.WORKLOADS["C2"], None, 1, sample_seqs=(0, 17, 63), paths=("gqa",))
    end_to_end(synth.WORKLOADS["C2"], None, 1, q_gain=4.0, sample_seqs=(5,), paths=("gqa", "absorb"))
    # the launch configuration bench.py times (balanced plan, two slots per sequence), every sequence, all
    # heads, both draft positions, on the peaked inputs
    end_to_end(synth.WORKLOADS["C2"], None, -2, q_gain=4.0, paths=("gqa",))


@pytest.mark.parametrize("s_q", [1, 2])
def test_c3_full_ragged(s_q):
    """Config 3: LLaMA-3-8B shape, B=128, seqlens uniform in [512, 32768]; both paths.
    The oracle runs the shortest, the longest and two more sequences."""
    from tests.parity_util import end_to_end
    w = synth.WORKLOADS["C3"].with_(s_q=s_q)
    sl = synth.make_seqlens(w)
    assert sl.min() >= 512 and sl.max() <= 32768
    sample = sorted({int(sl.argmin()), int(sl.argmax()), 3, 100})
    end_to_end(w, None, 4, q_gain=4.0, sample_seqs=sample)
    end_to_end(w, None, -3, q_gain=4.0, sample_seqs=sample)  # balanced plan: cuts inside long sequences


@pytest.mark.parametrize("s_q", [1, 2])
def test_c4_long_context_split_sweep(s_q):
    """Config 4: B=4, T=131072, split count swept over {1, 8, 32, 128} with the LSE combine."""
    from tests.parity_util import assert_close, dims_of
    from oracle import gqla_oracle as O
    from paper_2605_15250_b200.decoder import GqlaDecoder
    w = synth.WORKLOADS["C4"].with_(s_q=s_q)
    od, _ = dims_of(w)
    x = synth.make_inputs(w, q_gain=4.0)
    dec = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, x["w_uk"].cuda(), x["w_uv"].cuda(), x["cache"].cuda(),
                      x["seq_start"].cuda(), x["seqlens"].cuda(), w.scale)
    dec.expand_cache()
    b = 2  # the oracle runs one of the four sequences
    T = int(x["seqlens"][b])
    s0 = int(x["seq_start"][b])
    rows = synth.to_f64(x["cache"][s0:s0 + T])
    args = (od, synth.to_f64(x["q_c"][b:b + 1]), synth.to_f64(x["q_r"][b:b + 1]), synth.to_f64(x["w_uk"]),
            synth.to_f64(x["w_uv"]), rows, np.zeros(1, dtype=np.int64), np.array([T], dtype=np.int32), s_q, w.scale)
    ref_a = O.absorb_path(*args)
    ref_g = O.gqa_path(*args)
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().cuda()
    qc, qr = x["q_c"].cuda(), x["q_r"].cuda()
    for S in (1, 8, 32, 128, -32):
        a = dec.absorb_step(qc, qr, S).float().cpu().numpy()[b:b + 1]
        assert_close(a, ref_a, f"C4 absorb S={S}")
        gq = dec.gqa_step(q, S).float().cpu().numpy()[b:b + 1]
        assert_close(gq, ref_g, f"C4 gqa S={S}")
    dec.check_status()
