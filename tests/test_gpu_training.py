"""Training side of the layer on the GPU against the oracle: the mutual-information loss of the router (Eq. 4-6)
and the gradients of dense training (Eq. 3; Eq. 2 with a mask).  GPU required."""
import numpy as np
import pytest
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm
from harness import TOL_BF16, TOL_F32, Layer, desc_of, np_f32, record, rel_err, to_dev, to_np

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("T,E,zipf", [(1, 1, 0.0), (7, 3, 0.0), (300, 64, 1.1), (8192, 32, 0.0), (16384, 32, 1.1), (4099, 33, 0.0)])
def test_mi_loss_and_its_gradient(T, E, zipf):
    s = gi.LayerSpec(f"mi_{T}_{E}", T=T, d=128, H=64, E=E, dtype="bf16", router_gain=4.0, zipf_s=zipf)
    x, (Wr, br) = gi.tokens(s), gi.router(s)
    S = oracle.router_scores(x, Wr, br)
    L, He, Hc, grad = oracle.mi_loss(S, want_grad=True)
    desc = desc_of(s)
    ws = torch.empty(dm.dsmoe_workspace_size_stages(desc), dtype=torch.uint8, device="cuda")
    out3 = torch.zeros(3, dtype=torch.float32, device="cuda")
    g_d = torch.zeros((T, E), dtype=torch.float32, device="cuda")
    dm.dsmoe_mi_loss(desc, to_dev(S), out3, g_d, ws)
    got = out3.cpu().numpy().astype(np.float64)
    # sums in double on both sides; what is left is the rounding of the three results to fp32
    assert got[1] == pytest.approx(He, rel=2e-7, abs=1e-7) and got[2] == pytest.approx(Hc, rel=2e-7, abs=1e-7)
    assert got[0] == pytest.approx(L, abs=2e-7 * max(1.0, He))
    gg = g_d.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(gg - grad) <= 2e-7 * np.abs(grad) + 1e-12)
    record("mi_loss", T=T, E=E, L_MI=float(got[0]), H_e=float(got[1]), H_cond=float(got[2]), oracle_L_MI=L)
    out3b = torch.zeros(3, dtype=torch.float32, device="cuda")
    dm.dsmoe_mi_loss(desc, to_dev(S), out3b, None, ws)               # without the gradient; bit-identical
    assert torch.equal(out3, out3b)


def _backward_case(s, packed, masked, sample=None):
    L = Layer(s, pack=packed)
    dO = gi.normal(s.seed, f"{s.name}.dO", (s.T, s.d), 1.0, s.dtype)
    S = L.oracle_scores()
    mask = None
    if masked:
        mask, _ = oracle.select(S, oracle.MODE_TOPK, K=max(1, s.E // 3))
    dS = torch.zeros((s.T, s.E), dtype=torch.float32, device="cuda")
    dA = torch.zeros((s.T, s.E * s.H), dtype=L.native, device="cuda")
    dm.dsmoe_dense_backward(L.desc, L.x_d, L.W1_d, L.W2_d, L.packed, to_dev(S), to_dev(mask) if masked else None,
                            to_dev(dO), dS, dA, L.ws, L.dev_status)
    torch.cuda.synchronize()
    assert int(L.dev_status.item()) == 0
    ids = None if sample is None or sample >= s.T else gi.sample_tokens(s, sample)
    dS_ref, dA_ref = oracle.dense_backward(L.x, L.W1, L.W2, S, dO, mask=mask, token_ids=ids)
    dS_g = dS.cpu().numpy() if ids is None else dS.cpu().numpy()[ids]
    dA_g = np_f32(dA).reshape(s.T, s.E, s.H)
    dA_g = dA_g if ids is None else dA_g[ids]
    e_s = rel_err(dS_g, dS_ref)
    # dA is stored in the layer's type.  For bf16 that last rounding alone is up to 2^-9 of the value, more than the
    # whole tolerance for an element beyond 5 sigma, so it is allowed for separately: the bar is on
    # |dA - ref| - 2^-8 |ref| (the rounding of the stored value, with a factor 2 of slack), relative to RMS(ref)
    a_g, a_r = dA_g.reshape(len(dS_g), -1).astype(np.float64), dA_ref.reshape(len(dS_g), -1)
    slack = (2.0 ** -8) * np.abs(a_r) if s.dtype == "bf16" else 0.0
    rms = float(np.sqrt(np.mean(a_r ** 2)))
    e_a = float(np.max(np.maximum(np.abs(a_g - a_r) - slack, 0.0))) / max(rms, 1e-300)
    record("dense_backward", name=s.name, T=s.T, d=s.d, H=s.H, E=s.E, dtype=s.dtype, packed=bool(L.packed is not None),
           masked=masked, err_dS=e_s, err_dA=e_a, tokens_compared=int(len(dS_g)))
    if masked:
        M = np.array([[(int(m) >> e) & 1 for e in range(s.E)] for m in (mask if ids is None else mask[ids])], dtype=bool)
        assert np.all(dS_g[~M] == 0.0) and np.all(dA_g[~M] == 0.0)            # Eq. 2: nothing flows to inactive experts
    return e_s, e_a


BWD = [
    dict(T=64, d=256, H=512, E=8, dtype="f32"),
    dict(T=129, d=72, H=40, E=33, dtype="f32"),
    dict(T=33, d=128, H=136, E=5, dtype="bf16"),          # H % 64 != 0: plain kernel
    dict(T=300, d=128, H=64, E=64, dtype="bf16"),
    dict(T=260, d=320, H=192, E=8, dtype="bf16"),         # ragged column tiles
    dict(T=517, d=256, H=448, E=16, dtype="bf16"),
    dict(T=7, d=64, H=64, E=3, dtype="bf16"),
]


@pytest.mark.parametrize("masked", [False, True], ids=["dense", "masked"])
@pytest.mark.parametrize("packed", [False, True], ids=["plain", "packed"])
@pytest.mark.parametrize("case", BWD, ids=[str(i) for i in range(len(BWD))])
def test_dense_training_gradients(case, packed, masked):
    if packed and (case["dtype"] != "bf16" or case["H"] % 64 or case["d"] % 64):
        pytest.skip("packed weights: bf16, multiples of 64")
    s = gi.LayerSpec(f"bwd{BWD.index(case)}", router_gain=4.0, **case)
    e_s, e_a = _backward_case(s, packed, masked)
    tol = TOL_F32 if case["dtype"] == "f32" else TOL_BF16
    assert e_s <= tol and e_a <= tol, (e_s, e_a)


def test_dense_training_gradients_at_the_dense_forward_size():
    """T = 16384, d = 2048, 32 experts of width 1024 (the dense-training forward's benchmark shape), compared on 128
    seeded tokens (each token costs the oracle every expert twice over)."""
    s = gi.spec("c4")
    e_s, e_a = _backward_case(s, True, False, sample=128)
    assert e_s <= TOL_BF16 and e_a <= TOL_BF16, (e_s, e_a)
