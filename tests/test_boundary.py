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
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 0, p, p, 576, 10, p, p, p, p, None, None) == 2  # splits < 1
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 1, p, p, 576, 10, None, p, p, p, None, None) == 1
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 1, p, p, 100, 10, p, p, p, p, None, None) == 2
    assert L.gqla_decode_absorb(r(d), 0, 1, 1, 0.1, 1, odd, p, 576, 10, p, p, p, p, None, None) == 3
    assert L.gqla_decode_gqa(r(d), 0, 1, 1, 0.1, 1, p, p, p, p, 32, 10, p, p, p, p, None, None) == 2  # k_r stride < d_r
    assert L.gqla_decode_gqa(r(d), 0, 1, 1, 0.1, 1, p, None, p, p, 64, 10, p, p, p, p, None, None) == 1
    assert L.gqla_combine_splits(1, 128, 0, 512, 0, p, p, p, None, None) == 2
    assert L.gqla_combine_splits(1, 128, 4, 512, 0, p, None, p, None, None) == 1
    assert L.gqla_combine_splits(1, 128, 4, 512, 9, p, p, p, None, None) == 4
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
