"""The tensor-core GEMM kernel as CTA pairs (tcgen05 .cta_group::2: two CTAs share one 256-row tile), forced on every
launch whose shapes allow it -- the library itself pairs only where that was measured faster -- and compared with
the oracle on the grouped path with both aggregation modes, the dense forward, ragged column tiles, tiles whose
second half lies past the rows, and the backward pass (GPU required)."""
import os

import pytest

import dsmoe_inputs as gi
from harness import TOL_BF16, layer_parity, np_f32
from test_gpu_training import _backward_case

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def pairs_forced():
    old = os.environ.get("DSMOE_GEMM_PAIR")
    os.environ["DSMOE_GEMM_PAIR"] = "1"
    yield
    if old is None:
        del os.environ["DSMOE_GEMM_PAIR"]
    else:
        os.environ["DSMOE_GEMM_PAIR"] = old


PAIRED = [
    dict(T=2048, d=512, H=256, E=32, mode=gi.MODE_TOPK, K=6, fuse_combine=1),
    dict(T=2048, d=512, H=256, E=32, mode=gi.MODE_TOPK, K=6, fuse_combine=2),
    dict(T=300, d=448, H=320, E=8, mode=gi.MODE_TOPK, K=3, fuse_combine=1),        # ragged column tiles, 1 to 2 row tiles per expert
    dict(T=300, d=448, H=320, E=8, mode=gi.MODE_TOPK, K=3, fuse_combine=2),
    dict(T=1000, d=256, H=128, E=32, mode=gi.MODE_THRESHOLD, eps=0.7, eps_normalized=1, zipf_s=1.1, fuse_combine=1),   # empty and tiny experts
    dict(T=700, d=256, H=64, E=64, mode=gi.MODE_TOPK, K=64, fuse_combine=2),
    dict(T=260, d=320, H=192, E=8, mode=gi.MODE_ALL),                               # dense: 260 rows = one pair tile + 4 rows
    dict(T=1500, d=256, H=448, E=16, mode=gi.MODE_ALL, out_fp32=1),
    dict(T=513, d=128, H=128, E=16, mode=gi.MODE_THRESHOLD_TOPK, eps=0.03),
]


@pytest.mark.parametrize("case", PAIRED, ids=[str(i) for i in range(len(PAIRED))])
def test_layer_with_cta_pairs(case):
    s = gi.LayerSpec(f"pair{PAIRED.index(case)}", dtype="bf16", router_gain=4.0, **case)
    r = layer_parity(s)
    assert r["err_rows"] <= TOL_BF16, (r["err_rows"], r["err"])
    L = r["layer"]
    a = np_f32(L.forward()).copy()
    b = np_f32(L.forward())
    assert (a == b).all()                          # ordered sums: bit-identical from run to run


def test_full_size_prefill_with_cta_pairs():
    r = layer_parity(gi.spec("c3"), sample=256)
    assert r["err_rows"] <= TOL_BF16 and r["err"] <= TOL_BF16, (r["err_rows"], r["err"])


@pytest.mark.parametrize("masked", [False, True], ids=["dense", "masked"])
def test_backward_with_cta_pairs(masked):
    s = gi.LayerSpec("pair_bwd", T=517, d=256, H=448, E=16, dtype="bf16", router_gain=4.0)
    e_s, e_a = _backward_case(s, True, masked)
    assert e_s <= TOL_BF16 and e_a <= TOL_BF16, (e_s, e_a)
