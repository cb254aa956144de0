"""Group-axis sharding of the GQA path (Sec. 3.2): index arithmetic on the CPU, two gloo ranks that each
decode their groups with the oracle, and -- on a GPU -- the ranks' shards run one after another through
the library on one device."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import synth
from paper_2605_15250_b200.group_tp import GroupShard, gather_heads


def test_shards_partition_heads_and_groups():
    for h_q, g, world in ((128, 8, 1), (128, 8, 2), (128, 8, 8), (32, 8, 4), (28, 4, 2)):
        heads, groups = [], []
        for r in range(world):
            s = GroupShard(r, world, h_q, g)
            heads += list(range(h_q))[s.heads]
            groups += list(range(g))[s.groups]
            od = O.Dims(h_q, g, 128, 512, 64)
            # every head of the rank belongs to one of the rank's groups (the paper's j(i))
            assert {O.group_of_head(od, i) for i in range(h_q)[s.heads]} == set(range(g)[s.groups])
            # 2 g d_h / world + d_r elements per token (the shared RoPE key is the only replicated part)
            assert s.cache_elems_per_token(128, 64) == 2 * (g // world) * 128 + 64
        assert heads == list(range(h_q)) and groups == list(range(g))
    with pytest.raises(ValueError):
        GroupShard(0, 3, 128, 8)
    with pytest.raises(ValueError):
        GroupShard(2, 2, 128, 8)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs():
    w = synth.Workload("tp", 16, 4, 16, 32, 8, batch=3, s_q=2, dtype="f32", seed=0x77)
    return w, synth.make_inputs(w, seqlens=np.array([37, 0, 130], dtype=np.int32))


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w, x = _inputs()
        s = GroupShard(rank, world, w.h_q, w.g)
        f = {k: synth.to_f64(x[k]) for k in ("q_c", "q_r", "cache", "w_uk", "w_uv")}
        od = O.Dims(s.h_local, s.g_local, w.d_h, w.r_kv, w.d_r)
        o = O.gqa_path(od, f["q_c"][:, :, s.heads], f["q_r"][:, :, s.heads], f["w_uk"][s.groups], f["w_uv"][s.groups],
                       f["cache"], x["seq_start"].numpy(), x["seqlens"].numpy(), w.s_q, w.scale)
        mine = torch.from_numpy(np.ascontiguousarray(o))
        parts = [torch.empty_like(mine) for _ in range(world)]
        dist.all_gather(parts, mine)  # stands in for the layer's own exchange after W^O; not part of the path
        out.put((rank, gather_heads(parts).numpy()))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_unsharded_gqa_path():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((r, o) for r, o in (out.get(timeout=180) for _ in range(world)))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w, x = _inputs()
    f = {k: synth.to_f64(x[k]) for k in ("q_c", "q_r", "cache", "w_uk", "w_uv")}
    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    full = O.gqa_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], x["seq_start"].numpy(),
                      x["seqlens"].numpy(), w.s_q, w.scale)
    for _, o in res:
        assert np.allclose(o, full, rtol=0, atol=1e-12)


@pytest.mark.gpu
@pytest.mark.parametrize("world", [2, 8])
def test_shards_run_through_the_library_one_after_another(world):
    """One device stands in for `world` ranks, whose shards run one after another (no kernel waits for
    another): every rank expands and attends only its groups; the concatenated heads must match the
    oracle's unsharded GQA path, and -- with the fixed split plan, whose cut points do not depend on the
    number of groups -- the unsharded library run bit for bit."""
    from paper_2605_15250_b200 import binding as B
    from paper_2605_15250_b200 import build as gbuild
    from paper_2605_15250_b200.decoder import GqlaDecoder
    from paper_2605_15250_b200.group_tp import shard_decoder
    from tests.parity_util import assert_close
    gbuild.build()
    B.lib()
    w = synth.Workload("tp", 128, 8, 128, 512, 64, batch=4, s_q=2, dtype="bf16", seed=0x78)
    x = synth.make_inputs(w, seqlens=np.array([700, 1, 129, 2050], dtype=np.int32), q_gain=4.0)
    dev = torch.device("cuda", 0)
    cache, ss, sl = x["cache"].to(dev), x["seq_start"].to(dev), x["seqlens"].to(dev)
    w_uk, w_uv = x["w_uk"].to(dev), x["w_uv"].to(dev)
    q = torch.cat([x["q_c"], x["q_r"]], -1).contiguous().to(dev)
    whole = GqlaDecoder(w.h_q, w.g, w.d_h, w.r_kv, w.d_r, w_uk, w_uv, cache, ss, sl, w.scale)
    whole.expand_cache()
    o_whole = whole.gqa_step(q, 3).clone()
    parts, stored = [], 0
    for r in range(world):
        s = GroupShard(r, world, w.h_q, w.g)
        dec = shard_decoder(s, w.d_h, w.r_kv, w.d_r, w_uk, w_uv, cache, ss, sl, w.scale)
        dec.expand_cache()
        assert dec.k_c.shape == (cache.shape[0], s.g_local, w.d_h)
        stored += dec.k_c.numel() + dec.v.numel()
        parts.append(dec.gqa_step(s.slice_queries(q), 3).clone())
        dec.check_status()
    torch.cuda.synchronize()
    assert stored == whole.k_c.numel() + whole.v.numel()  # no K/V element is held twice across the ranks
    o = gather_heads(parts)
    assert torch.equal(o, o_whole)
    f = {k: synth.to_f64(x[k]) for k in ("q_c", "q_r", "cache", "w_uk", "w_uv")}
    od = O.Dims(w.h_q, w.g, w.d_h, w.r_kv, w.d_r)
    ref = O.gqa_path(od, f["q_c"], f["q_r"], f["w_uk"], f["w_uv"], f["cache"], x["seq_start"].numpy(), x["seqlens"].numpy(),
                     w.s_q, w.scale)
    assert_close(o.float().cpu().numpy(), ref, "group-sharded gqa path")
