"""Stage-by-stage parity of the C-ABI entry points against the CPU oracle (GPU required)."""
import numpy as np
import pytest
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm
from harness import (TOL_BF16, TOL_F32, Layer, desc_of, np_f32, rel_err, to_dev, to_np)

pytestmark = pytest.mark.gpu

SHAPES = [
    # name, T, d, H, E, dtype
    ("tiny", 64, 256, 512, 8, "f32"),
    ("odd", 129, 72, 40, 33, "f32"),
    ("one", 1, 64, 64, 1, "bf16"),
    ("e64", 300, 128, 64, 64, "bf16"),
    ("e3", 7, 64, 128, 3, "bf16"),
    ("mid", 517, 256, 136, 32, "bf16"),
]


def _spec(name, T, d, H, E, dtype, **kw):
    return gi.LayerSpec(f"st_{name}", T=T, d=d, H=H, E=E, dtype=dtype, router_gain=4.0, **kw)


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_router_scores(shape):
    s = _spec(*shape, zipf_s=1.1 if shape[0] in ("odd", "e64") else 0.0)
    x, (Wr, br) = gi.tokens(s), gi.router(s)
    scores = torch.empty((s.T, s.E), dtype=torch.float32, device="cuda")
    dm.dsmoe_router(desc_of(s), to_dev(x), to_dev(Wr), to_dev(br), scores)
    S_gpu, S_ref = scores.cpu().numpy(), oracle.router_scores(x, Wr, br)
    assert np.all(np.abs(S_gpu - S_ref) <= 1e-6 + 1e-5 * S_ref)


MODES = [
    dict(mode=gi.MODE_THRESHOLD, eps=0.02),
    dict(mode=gi.MODE_THRESHOLD, eps=0.48, eps_normalized=1),
    dict(mode=gi.MODE_THRESHOLD, eps=0.6, min_k=1),
    dict(mode=gi.MODE_THRESHOLD, eps=0.0),
    dict(mode=gi.MODE_TOPK, K=1),
    dict(mode=gi.MODE_TOPK, K=5),
    dict(mode=gi.MODE_TOPK, K=100),
    dict(mode=gi.MODE_ALL),
    dict(mode=gi.MODE_THRESHOLD_TOPK, eps=0.02),                          # Threshold-TopK: K from the batch
    dict(mode=gi.MODE_THRESHOLD_TOPK, eps=0.9, eps_normalized=1),
    dict(mode=gi.MODE_THRESHOLD_TOPK, eps=2.0),                           # nothing passes: K = 1
]


@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
@pytest.mark.parametrize("mode", MODES, ids=[str(i) for i in range(len(MODES))])
def test_select_and_permute_bit_exact_on_oracle_scores(shape, mode):
    s = _spec(*shape, **mode)
    desc = desc_of(s)
    x, (Wr, br) = gi.tokens(s), gi.router(s)
    S = oracle.router_scores(x, Wr, br)
    if shape[0] == "e3":                     # plant exact ties and exact threshold hits
        S[0, :] = np.float32(1 / 3)
        S[1, :] = np.float32([0.02, 0.02, 0.96])
    mask_ref, k_ref = oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
    W = dm.width(desc)
    g = oracle.group(mask_ref, S, width=W)
    ws = torch.empty(dm.dsmoe_workspace_size(desc), dtype=torch.uint8, device="cuda")
    S_d = to_dev(S)
    mask = torch.zeros(s.T, dtype=torch.int64, device="cuda")
    k_t = torch.zeros(s.T, dtype=torch.int32, device="cuda")
    counts = torch.full((s.E,), -7, dtype=torch.int32, device="cuda")
    offsets = torch.full((s.E + 1,), -7, dtype=torch.int32, device="cuda")
    dm.dsmoe_select(desc, S_d, mask, k_t, counts, offsets, ws)
    assert np.array_equal(to_np(mask).view(np.uint64), mask_ref)
    assert np.array_equal(to_np(k_t), k_ref)
    assert np.array_equal(to_np(counts), g["counts"])
    assert np.array_equal(to_np(offsets), g["offsets"])
    amax = dm.amax(desc)
    row_token = torch.full((amax,), -9, dtype=torch.int32, device="cuda")
    row_gate = torch.zeros(amax, dtype=torch.float32, device="cuda")
    token_rows = torch.full((s.T, W), -9, dtype=torch.int32, device="cuda")
    x_d = to_dev(x)
    xp = torch.zeros((amax, s.d), dtype=x_d.dtype, device="cuda")
    dm.dsmoe_permute(desc, x_d, S_d, mask, offsets, row_token, row_gate, token_rows, xp, ws)
    A = g["A"]
    assert np.array_equal(to_np(row_token)[:A], g["row_token"])
    assert np.all(to_np(row_token)[A:] == -9)                       # nothing written past A
    assert np.array_equal(to_np(row_gate)[:A], g["row_gate"])
    assert np.array_equal(to_np(token_rows), g["token_rows"])
    assert np.array_equal(to_np(xp)[:A], x[g["row_token"]])


@pytest.mark.parametrize("pack", [False, True], ids=["plain", "packed"])
@pytest.mark.parametrize("shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_expert_mlp_and_combine(shape, pack):
    s = _spec(*shape, mode=gi.MODE_TOPK, K=3)
    if pack and s.dtype != "bf16":
        pytest.skip("packed weights are bf16 only")
    desc = desc_of(s)
    L = Layer(s, pack=pack)
    S = L.oracle_scores()
    mask_ref, k_ref = L.oracle_select(S)
    W = dm.width(desc)
    g = oracle.group(mask_ref, S, width=W)
    A, amax = g["A"], dm.amax(desc)
    xp_np = np.zeros((amax, s.d), dtype=L.x.dtype)
    xp_np[:A] = L.x[g["row_token"]]
    xp = to_dev(xp_np)
    yp = torch.zeros((amax, s.d), dtype=xp.dtype, device="cuda")
    dm.dsmoe_expert_mlp(desc, xp, L.W1_d, L.W2_d, L.packed, to_dev(g["offsets"]), yp, L.ws, L.dev_status)
    torch.cuda.synchronize()
    assert int(L.dev_status.item()) == 0
    yp_ref = oracle.expert_rows(xp_np[:A], L.W1, L.W2, g["row_expert"])
    tol = TOL_BF16 if s.dtype == "bf16" else TOL_F32
    assert rel_err(np_f32(yp)[:A], yp_ref) <= tol
    # aggregation on the GPU's own yp against the oracle's aggregation of the same values
    out = torch.empty((s.T, s.d), dtype=xp.dtype, device="cuda")
    gate = np.zeros(amax, np.float32)
    gate[:A] = g["row_gate"]
    dm.dsmoe_combine(desc, yp, to_dev(gate), to_dev(g["token_rows"]), to_dev(k_ref), out)
    ref = oracle.combine(np_f32(yp), gate, g["token_rows"])
    rms = float(np.sqrt(np.mean(ref ** 2)))
    rtol = 2.0 ** -8 if s.dtype == "bf16" else 1e-6          # one rounding of the fp32 sum to the output type
    assert np.all(np.abs(np_f32(out) - ref) <= rtol * np.abs(ref) + 1e-6 * rms)
