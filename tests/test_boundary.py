"""Host-side checks of the C-ABI library that need no GPU: the symbols the header
declares are exported, the integer bookkeeping equals the oracle's, and argument
violations return a code before anything is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import gqla_oracle as O
from paper_2605_15250_b200 import binding as B
from paper_2605_15250_b200 import build as gbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


def _declared():
    names = []
    for fn in sorted(os.listdir(os.path.join(ROOT, "include"))):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names += re.findall(r"\b(gqla_[a-z0-9_]+)\s*\(", text)
    return sorted(set(names))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert {"gqla_absorb_q", "gqla_decode_absorb", "gqla_expand_cache", "gqla_decode_gqa", "gqla_combine_splits",
            "gqla_up_proj"} <= set(names)
    handle = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(handle, n), n
    assert set(names) == set(B.exported_symbols())


def test_split_plan_matches_oracle():
    rng = np.random.default_rng(7)
    cases = [(0, 1), (0, 5), (1, 1), (63, 2), (64, 2), (65, 2), (4096, 8), (131072, 128), (131072, 1), (100, 8)]
    cases += [(int(rng.integers(0, 140000)), int(rng.integers(1, 200))) for _ in range(300)]
    for T, S in cases:
        assert B.gqla_split_plan(T, S) == O.split_plan(T, S), (T, S)


def test_balanced_plan_matches_oracle():
    """The library's balanced split plan (walked worker by worker, as its kernels do) against the
    oracle's tile-by-tile statement of the same rule: ragged batches, empty sequences, more workers
    than tiles, a single worker, and the smallest slot count."""
    rng = np.random.default_rng(11)
    cases = [([4096] * 64, 3, 74), ([4096] * 64, 2, 18), ([0, 0, 0], 2, 5), ([1], 2, 148), ([0, 129, 0, 128, 0], 2, 3),
             ([131072] * 4, 8, 74), ([131072] * 4, 2, 18), ([5000, 0, 0], 4, 1), ([], 2, 4)]
    for _ in range(300):
        n = int(rng.integers(1, 40))
        sl = [int(x) for x in rng.integers(0, 40000, size=n)]
        for i in rng.integers(0, n, size=n // 4):
            sl[int(i)] = 0
        cases.append((sl, int(rng.integers(2, 9)), int(rng.integers(1, 160))))
    for sl, S, W in cases:
        plans, owners = B.gqla_balanced_plan(sl, S, W)
        assert plans == O.balanced_plan(sl, S, W), (sl, S, W)
        # the owner of a piece is the worker whose share holds its tiles; shares do not exceed `share`
        load = {}
        for b, T in enumerate(sl):
            for k, (lo, hi) in enumerate(plans[b]):
                if hi > lo:
                    assert owners[b][k] >= 0
                    load[owners[b][k]] = load.get(owners[b][k], 0) + -(-(hi - lo) // 128)
                else:
                    assert owners[b][k] == -1
        tiles = [-(-t // 128) for t in sl]
        share = max(-(-sum(tiles) // W), -(-max(tiles + [0]) // (S - 1)), 1)
        assert all(v <= share for v in load.values())
    assert B.lib().gqla_balanced_plan(None, 1, 2, 1, None, None, None) == 1
    buf = (ctypes.c_int32 * 8)()
    assert B.lib().gqla_balanced_plan(buf, 2, 1, 4, buf, buf, None) == 2  # fewer than two slots


def test_group_map_and_mask_limit_match_oracle():
    for h_q, g in ((128, 8), (32, 8), (8, 2), (28, 4), (20, 4), (64, 64), (7, 1)):
        d = B.make_dims(h_q, g, 128, 512, 64)
        od = O.Dims(h_q, g, 128, 512, 64)
        assert [B.gqla_group_of_head(d, i) for i in range(h_q)] == [O.group_of_head(od, i) for i in range(h_q)]
        assert B.gqla_group_of_head(d, h_q) == -1 and B.gqla_group_of_head(d, -1) == -1
    for T in (0, 1, 2, 3, 64, 4096):
        for s_q in (1, 2, 3, 4):
            for p in range(s_q):
                assert B.gqla_visible_limit(T, s_q, p) == O.visible_limit(T, s_q, p)


def test_argument_errors_return_before_launch():
    L = B.lib()
    d = B.make_dims(128, 8, 128, 512, 64)
    bad = B.make_dims(128, 7, 128, 512, 64)  # h_q % g != 0
    p = ctypes.c_void_p(0x1000)  # aligned, never dereferenced on these paths
    odd = ctypes.c_void_p(0x1004)
    r = ctypes.byref
    assert L.gqla_absorb_q(None, 0, 1, 1, p, p, p, p, None) == 1
    assert L.gqla_absorb_q(r(bad), 0, 1, 1, p, p, p, p, None) == 2
    assert L.gqla_absorb_q(r(d), 7, 1, 1, p, p, p, p, None) == 4
    assert L.gqla_absorb_q(r(d), 0, 1, 1, None, p, p, p, None) == 1
    assert L.gqla_absorb_q(r(d), 0, 1, 1, odd, p, p, p, None) == 3
    assert L.gqla_absorb_q(r(d), 0, -1, 1, p, p, p, p, None) == 2
    assert L.gqla_absorb_q(r(d), 0, 0, 1, p, p, p, p, None) == 0  # empty batch: nothing to do
    assert L.gqla_up_proj(r(d), 0, 1, 0, p, p, p, None) == 2
    assert L.gqla_up_proj(r(d), 0, 1, 1, p, None, p, None) == 1
    assert L.gqla_expand_cache(r(d), 0, 10, p, 575, p, p, p, p, p, None) == 2  # stride < r_kv + d_r
    assert L.gqla_expand_cache(r(d), 0, 10, p, 576, p, p, None, p, p, None) == 1
    assert L.gqla_expand_cache(r(d), 0, 0, None, 576, None, None, None, None, None, None) == 0
    assert L.gqla_append_expand(r(d), 0, 4, 0, p, 576, p, p, p, p, p, p, p, None) == 2  # s_q < 1
    assert L.gqla_append_expand(r(d), 0, 4, 1, p, 575, p, p, p, p, p, p, p, None) == 2  # stride < r_kv + d_r
    assert L.gqla_append_expand(r(d), 0, 4, 1, p, 576, p, None, p, p, p, p, p, None) == 1
    assert L.gqla_append_expand(r(d), 0, 4, 1, p, 576, p, p, p, p, odd, p, p, None) == 3
    assert L.gqla_append_expand(r(d), 0, 0, 1, None, 576, None, None, None, None, None, None, None, None) == 0
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 0, p, p, 576, 10, p, p, p, p, None, None) == 2  # splits < 1
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 1, p, p, 576, 10, None, p, p, p, None, None) == 1
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 1, p, p, 100, 10, p, p, p, p, None, None) == 2
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 1, odd, p, 576, 10, p, p, p, p, None, None) == 3
    assert L.gqla_decode_absorb_final(r(d), 0, 1, 0, 0.1, p, p, 576, 10, p, p, p, None, None, None) == 2  # s_q < 1
    assert L.gqla_decode_absorb_final(r(d), 0, 1, 1, 0.1, p, p, 576, 10, p, p, None, None, None, None) == 1
    assert L.gqla_decode_absorb_final(r(d), 0, 1, 1, 0.1, p, p, 576, 10, p, p, odd, None, None, None) == 3
    assert L.gqla_decode_absorb_final(r(d), 0, 1, 1, 0.1, p, p, 100, 10, p, p, p, None, None, None) == 2
    assert L.gqla_decode_absorb_final(r(d), 0, 0, 1, 0.1, None, None, 576, 0, None, None, None, None, None, None) == 0
    assert L.gqla_decode_absorb_paged(r(d), 0, 1, 1, 0.1, 1, p, p, 576, 10, None, 4, 128, p, p, p, None, None) == 1
    assert L.gqla_decode_absorb_paged(r(d), 0, 1, 1, 0.1, 1, p, p, 576, 10, p, 4, 0, p, p, p, None, None) == 2  # page size
    assert L.gqla_decode_absorb_paged(r(d), 0, 1, 1, 0.1, 1, p, p, 576, 10, p, 0, 128, p, p, p, None, None) == 2
    assert L.gqla_decode_gqa_paged(r(d), 0, 1, 1, 0.1, 1, p, p, p, p, 64, 10, None, 4, 128, p, p, p, None, None) == 1
    assert L.gqla_decode_gqa_paged(r(d), 0, 1, 1, 0.1, -1, p, p, p, p, 64, 10, p, 4, 128, p, p, p, None, None) == 2
    assert L.gqla_decode_gqa_paged(r(d), 0, 0, 1, 0.1, 1, None, None, None, None, 64, 0, None, 4, 128, None, None, None,
                                   None, None) == 0
    assert L.gqla_decode_gqa(r(d), 0, 1, 1, 0.1, 1, p, p, p, p, 32, 10, p, p, p, p, None, None) == 2  # k_r stride < d_r
    assert L.gqla_decode_gqa(r(d), 0, 1, 1, 0.1, 1, p, None, p, p, 64, 10, p, p, p, p, None, None) == 1
    assert L.gqla_combine_splits(1, 128, 0, 512, 0, p, p, p, None, None) == 2
    assert L.gqla_combine_splits(1, 128, 4, 512, 0, p, None, p, None, None) == 1
    assert L.gqla_combine_splits(1, 128, 4, 512, 9, p, p, p, None, None) == 4
    assert L.gqla_combine_up_proj(r(d), 0, 1, 1, 0, p, p, p, p, None, None) == 2  # splits < 1
    assert L.gqla_combine_up_proj(r(d), 0, 1, 1, 2, p, None, p, p, None, None) == 1
    assert L.gqla_combine_up_proj(r(d), 0, 1, 1, 2, p, p, odd, p, None, None) == 3
    assert B.lib().gqla_status_str(3).decode().startswith("pointer")


def test_policy_switch_and_kernel_names():
    d = B.make_dims(8, 2, 16, 32, 8)
    B.set_policy(B.POLICY_GENERIC)
    assert B.get_policy() == B.POLICY_GENERIC
    import torch
    assert B.kernel_for(d, torch.float32, 1, "absorb") == "generic"
    B.set_policy(B.POLICY_AUTO)
    assert B.get_policy() == B.POLICY_AUTO
    # fp32 storage is never on the tensor-core kernels
    assert B.kernel_for(d, torch.float32, 1, "gqa") == "generic"


def test_status_word_registration_round_trips():
    """The process-wide status word of the projection calls: what is registered is what the library
    hands to its kernels, and NULL unregisters.  Nothing is launched and the address is never dereferenced."""
    L = B.lib()
    assert B.get_status_word() == 0
    L.gqla_set_status_word(ctypes.c_void_p(0x7000))
    try:
        assert B.get_status_word() == 0x7000
    finally:
        L.gqla_set_status_word(None)
    assert B.get_status_word() == 0
