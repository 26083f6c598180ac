"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, validates arguments, and sizes its workspace sensibly."""
import ctypes
import os
import re

import pytest

import paper_2404_05567_b200 as dm
from paper_2404_05567_b200 import build as dm_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    dm_build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "dsmoe.h")).read()
    declared = set(re.findall(r"\b(dsmoe_[a-z_]+)\s*\(", header))
    assert declared == set(dm.EXPORTS)
    L = ctypes.CDLL(dm.binding.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings():
    assert dm.status_string(0) == "ok"
    assert "workspace" in dm.status_string(3)
    assert dm.status_string(99) == "unknown status"


def test_desc_validation_and_workspace_size():
    good = dm.make_desc(64, 256, 512, 8, dm.F32, dm.SELECT_THRESHOLD, eps=0.1)
    n = dm.dsmoe_workspace_size(good)
    # at least scores + grouped copies of the tokens and expert outputs
    assert n >= 64 * 8 * 4 + 2 * 64 * 8 * 256 * 4
    bad = [
        dict(E=65), dict(E=0), dict(d=12), dict(H=4), dict(T=-1), dict(dtype=7), dict(mode=5),
        dict(mode=dm.SELECT_TOPK, K=0), dict(min_k=2), dict(eps=float("nan")),
    ]
    for kw in bad:
        args = dict(T=64, d=256, H=512, E=8, dtype=dm.F32, mode=dm.SELECT_THRESHOLD, eps=0.1)
        args.update(kw)
        with pytest.raises(dm.DsmoeError) as ei:
            dm.dsmoe_workspace_size(dm.make_desc(**args))
        assert ei.value.code in (1, 2)
    with pytest.raises(dm.DsmoeError) as ei:
        dm.dsmoe_workspace_size(dm.make_desc(8, 64, 64, 65))
    assert ei.value.code == 2                      # E > 64 is "unsupported", not "invalid"
    topk = dm.make_desc(128, 64, 64, 32, dm.BF16, dm.SELECT_TOPK, K=4)
    thr = dm.make_desc(128, 64, 64, 32, dm.BF16, dm.SELECT_THRESHOLD)
    assert dm.dsmoe_workspace_size(topk) < dm.dsmoe_workspace_size(thr)   # Amax = T*K vs T*E
    assert dm.amax(topk) == 128 * 4 and dm.amax(thr) == 128 * 32


def test_null_pointers_and_short_workspace_are_rejected_before_any_launch():
    desc = dm.make_desc(4, 64, 64, 4, dm.F32)
    L = dm.lib()
    z = ctypes.c_void_p(0)
    assert L.dsmoe_router(ctypes.byref(desc), z, z, z, z, z) == 1
    assert L.dsmoe_layer_forward(ctypes.byref(desc), z, z, z, z, z, z, z, z, z, z, ctypes.c_size_t(0), z, z) == 1
    fake = ctypes.c_void_p(4096)                   # aligned, never dereferenced on the host
    assert L.dsmoe_layer_forward(ctypes.byref(desc), fake, fake, z, fake, fake, z, fake, z, z, fake,
                                 ctypes.c_size_t(16), z, z) == 3
    odd = ctypes.c_void_p(4100)
    assert L.dsmoe_layer_forward(ctypes.byref(desc), odd, fake, z, fake, fake, z, fake, z, z, fake,
                                 ctypes.c_size_t(1 << 30), z, z) == 1
    # packed weights only exist for bf16
    assert L.dsmoe_packed_size(ctypes.byref(desc), ctypes.byref(ctypes.c_size_t(0))) == 1
    empty = dm.make_desc(0, 64, 64, 4, dm.F32)
    assert L.dsmoe_layer_forward(ctypes.byref(empty), z, z, z, z, z, z, z, z, z, z, ctypes.c_size_t(0), z, z) == 0
    # the host-buffer forms: a missing host or staging buffer is rejected before any copy; T = 0 is a no-op
    for fn in (L.dsmoe_layer_forward_host, L.dsmoe_layer_forward_host_async):
        assert fn(ctypes.byref(desc), z, fake, z, z, fake, fake, z, fake, fake, fake, ctypes.c_size_t(1 << 30), z, z) == 1
        assert fn(ctypes.byref(desc), fake, fake, z, z, fake, fake, z, fake, z, fake, ctypes.c_size_t(1 << 30), z, z) == 1
        assert fn(ctypes.byref(empty), z, z, z, z, z, z, z, z, z, z, ctypes.c_size_t(0), z, z) == 0


def test_pack_rejects_shapes_that_are_not_multiples_of_64_and_the_new_selection_mode_is_accepted():
    L = dm.lib()
    fake = ctypes.c_void_p(4096)
    z = ctypes.c_void_p(0)
    odd = dm.make_desc(16, 128, 72, 4, dm.BF16)          # H = 72: the packed layout is in blocks of 64
    assert L.dsmoe_pack_weights(ctypes.byref(odd), fake, fake, fake, z) == 2
    # Threshold-TopK is a valid mode of the descriptor (sizes as for the threshold rule: up to E experts per token) ...
    tt = dm.make_desc(128, 64, 64, 32, dm.BF16, mode=dm.SELECT_THRESHOLD_TOPK, eps=0.1)
    thr = dm.make_desc(128, 64, 64, 32, dm.BF16, mode=dm.SELECT_THRESHOLD, eps=0.1)
    assert dm.dsmoe_workspace_size(tt) >= dm.dsmoe_workspace_size(thr) - 4096 and dm.amax(tt) == 128 * 32
    # ... a mode beyond it is not
    bad = dm.make_desc(128, 64, 64, 32, dm.BF16, mode=4)
    assert L.dsmoe_workspace_size(ctypes.byref(bad), ctypes.byref(ctypes.c_size_t(0))) == 1
