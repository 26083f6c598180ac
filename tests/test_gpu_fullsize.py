"""Parity at the benchmark workloads' full sizes and in the corners the smaller cases do not reach (GPU required):
selection, counts, offsets and permutation indices bit-exact against the oracle on the oracle's own scores; tile
widths that need more than one weight copy; the device-side check of corrupt expert segments; the selection
statistics."""
import numpy as np
import pytest
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm
from harness import (TOL_BF16, Layer, desc_of, layer_parity, np_f32, record, rel_err, to_dev, to_np)

pytestmark = pytest.mark.gpu

FULL = [("c3", {}), ("c4", {})] + [("c5", dict(eps=e)) for e in (0.0, 0.01, 0.05, 0.1, 0.2)]


@pytest.mark.parametrize("cfg,kw", FULL, ids=["c3", "c4"] + [f"c5_eps{e}" for e in (0.0, 0.01, 0.05, 0.1, 0.2)])
def test_full_size_select_and_permute_bit_exact_on_oracle_scores(cfg, kw):
    """T = 8192 / 16384 / 4096: several rounds of the chunk scan (more than 128 chunks of 32 tokens)."""
    s = gi.spec(cfg, **kw)
    desc = desc_of(s)
    x, (Wr, br) = gi.tokens(s), gi.router(s)
    S = oracle.router_scores(x, Wr, br)
    mask_ref, k_ref = oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
    W = dm.width(desc)
    g = oracle.group(mask_ref, S, width=W)
    ws = torch.empty(dm.dsmoe_workspace_size_stages(desc), dtype=torch.uint8, device="cuda")
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
    amax, A = dm.amax(desc), g["A"]
    row_token = torch.full((amax,), -9, dtype=torch.int32, device="cuda")
    row_gate = torch.zeros(amax, dtype=torch.float32, device="cuda")
    token_rows = torch.full((s.T, W), -9, dtype=torch.int32, device="cuda")
    x_d = to_dev(x)
    xp = torch.zeros((amax, s.d), dtype=x_d.dtype, device="cuda")
    dm.dsmoe_permute(desc, x_d, S_d, mask, offsets, row_token, row_gate, token_rows, xp, ws)
    assert np.array_equal(to_np(row_token)[:A], g["row_token"])
    assert np.all(to_np(row_token)[A:] == -9)
    assert np.array_equal(to_np(row_gate)[:A], g["row_gate"])
    assert np.array_equal(to_np(token_rows), g["token_rows"])
    # the grouped copy of the tokens, checked on the device against an index by the oracle's row list
    rt = torch.from_numpy(g["row_token"].astype(np.int64)).cuda()
    assert torch.equal(xp[:A].view(torch.int16), x_d[rt].view(torch.int16))
    # the selection statistics of the same call
    st_d = torch.zeros(288, dtype=torch.uint8, device="cuda")
    dm.dsmoe_stats(desc, S_d, mask, st_d)
    st = dm.read_stats(st_d)
    assert st["assignments"] == A and st["counts"][:s.E] == g["counts"].tolist()
    assert st["zero_tokens"] == int((mask_ref == 0).sum()) and st["empty_experts"] == int((g["counts"] == 0).sum())
    near = 0
    if s.mode == gi.MODE_THRESHOLD:
        v = (S * np.float32(s.E)) if s.eps_normalized else S
        near = int((np.abs(v.astype(np.float64) - float(np.float32(s.eps))) <= 1e-6).sum())
    assert st["near_threshold"] == near
    record("selection_stats", name=s.name, eps=s.eps, A=A, zero_tokens=st["zero_tokens"], empty_experts=st["empty_experts"],
           near_threshold=near)


# Tile widths that are not 64, 128 or 256: a ragged last column tile of 192 (= 128 + 64) or 64 rows after one or two
# full tiles, on the grouped (sparse prefill), the dense and the decode path.
ODD = [dict(d=320, H=192), dict(d=448, H=320), dict(d=192, H=448), dict(d=704, H=448)]


@pytest.mark.parametrize("shape", ODD, ids=[f"d{o['d']}_H{o['H']}" for o in ODD])
@pytest.mark.parametrize("path", ["grouped", "dense", "decode"])
def test_tile_widths_that_need_several_weight_copies(shape, path):
    kw = dict(grouped=dict(T=300, mode=gi.MODE_TOPK, K=3), dense=dict(T=260, mode=gi.MODE_ALL),
              decode=dict(T=20, mode=gi.MODE_TOPK, K=3))[path]
    s = gi.LayerSpec(f"odd_{path}", E=8, dtype="bf16", router_gain=4.0, **shape, **kw)
    r = layer_parity(s)
    assert r["err_rows"] <= TOL_BF16 and r["err"] <= TOL_BF16, (r["err_rows"], r["err"])


def _grouped_inputs(s):
    L = Layer(s)
    S = L.oracle_scores()
    mask_ref, _ = L.oracle_select(S)
    g = oracle.group(mask_ref, S, width=dm.width(L.desc))
    A, amax = g["A"], dm.amax(L.desc)
    xp_np = np.zeros((amax, s.d), dtype=L.x.dtype)
    xp_np[:A] = L.x[g["row_token"]]
    return L, g, to_dev(xp_np), A, amax


def test_corrupt_expert_segments_are_reported_and_never_written():
    """Segments that are negative, decreasing or end beyond Amax: the kernel treats that expert as empty and writes
    DSMOE_ERR_INVALID_ARG to *dev_status; every other expert's rows come out as usual."""
    s = gi.LayerSpec("badoff", T=300, d=128, H=128, E=8, dtype="bf16", mode=gi.MODE_TOPK, K=2, router_gain=4.0)
    L, g, xp, A, amax = _grouped_inputs(s)
    good = torch.full((amax, s.d), 7.0, dtype=torch.bfloat16, device="cuda")
    dm.dsmoe_expert_mlp(L.desc, xp, L.W1_d, L.W2_d, L.packed, to_dev(g["offsets"]), good, L.ws, L.dev_status)
    torch.cuda.synchronize()
    assert int(L.dev_status.item()) == 0
    off = g["offsets"].copy()
    cases = [
        # (edit, rows that may differ from the good run, rows that must stay untouched)
        (lambda o: o.__setitem__(s.E, amax + 1), (int(off[s.E - 1]), A), (int(off[s.E - 1]), A)),   # last expert ends beyond the buffers
        (lambda o: o.__setitem__(0, -3), (0, int(off[1])), (0, int(off[1]))),                        # first expert starts before them
        # expert 3 ends before it starts (empty); expert 4 then starts one row early and covers expert 3's rows
        (lambda o: o.__setitem__(4, int(o[3]) - 1), (int(off[3]) - 1, int(off[4])), None),
    ]
    for edit, (lo, hi), untouched in cases:
        bad = off.copy()
        edit(bad)
        yp = torch.full((amax, s.d), 7.0, dtype=torch.bfloat16, device="cuda")
        L.dev_status.zero_()
        dm.dsmoe_expert_mlp(L.desc, xp, L.W1_d, L.W2_d, L.packed, to_dev(bad), yp, L.ws, L.dev_status)
        torch.cuda.synchronize()
        assert int(L.dev_status.item()) == 1                                      # DSMOE_ERR_INVALID_ARG
        touched = (yp != 7.0).any(dim=1).cpu().numpy()
        same = (yp == good).all(dim=1).cpu().numpy()
        outside = np.ones(amax, bool)
        outside[lo:hi] = False
        assert same[outside].all()                                                # every other expert's rows as usual
        if untouched is not None:
            assert not touched[untouched[0]:untouched[1]].any()


def test_permute_skips_rows_that_inconsistent_offsets_would_put_out_of_range():
    s = gi.LayerSpec("badperm", T=200, d=64, H=64, E=8, dtype="bf16", mode=gi.MODE_TOPK, K=2, router_gain=4.0)
    L, g, _, A, amax = _grouped_inputs(s)
    S = L.oracle_scores()
    mask_ref, _ = L.oracle_select(S)
    bad = g["offsets"].copy()
    bad[s.E - 1] = amax - 1                  # the last expert's rows would start at the buffer's last row
    row_token = torch.full((amax + 64,), -9, dtype=torch.int32, device="cuda")     # 64 guard entries behind the buffer
    row_gate = torch.zeros(amax + 64, dtype=torch.float32, device="cuda")
    token_rows = torch.full((s.T, 2), -9, dtype=torch.int32, device="cuda")
    xp = torch.zeros((amax, s.d), dtype=torch.bfloat16, device="cuda")
    dm.dsmoe_permute(L.desc, L.x_d, to_dev(S), to_dev(mask_ref), to_dev(bad), row_token, row_gate, token_rows, xp, L.ws)
    torch.cuda.synchronize()
    assert np.all(to_np(row_token)[amax:] == -9)


# ---------------------------------------------------------------- where the aggregation runs: inside the down-projection
# (fuse_combine = 1) or as a second kernel over fp32 gate-weighted rows (2); 0 lets the library choose by H

FUSED = [
    dict(T=300, d=64, H=64, E=16, mode=gi.MODE_THRESHOLD, eps=0.5),                      # most tokens select nothing
    dict(T=300, d=64, H=64, E=16, mode=gi.MODE_THRESHOLD, eps=0.5, min_k=1),
    dict(T=1000, d=256, H=128, E=32, mode=gi.MODE_THRESHOLD, eps=0.7, eps_normalized=1, zipf_s=1.1),
    dict(T=2048, d=512, H=256, E=32, mode=gi.MODE_TOPK, K=6),                            # several row tiles per expert
    dict(T=300, d=448, H=320, E=8, mode=gi.MODE_TOPK, K=3),                              # ragged column tiles
    dict(T=700, d=256, H=64, E=64, mode=gi.MODE_TOPK, K=64),                             # every expert, grouped
    dict(T=513, d=128, H=128, E=16, mode=gi.MODE_THRESHOLD_TOPK, eps=0.03),
    dict(T=260, d=128, H=128, E=8, mode=gi.MODE_TOPK, K=2, out_fp32=1),
]


@pytest.mark.parametrize("fuse", [1, 2], ids=["inside", "separate"])
@pytest.mark.parametrize("case", FUSED, ids=[str(i) for i in range(len(FUSED))])
def test_aggregation_inside_the_down_projection(case, fuse):
    s = gi.LayerSpec(f"fused{FUSED.index(case)}", dtype="bf16", router_gain=5.0, fuse_combine=fuse, **case)
    r = layer_parity(s)
    assert r["err_rows"] <= TOL_BF16, (r["err_rows"], r["err"])
    L = r["layer"]
    a = np_f32(L.forward()).copy()
    b = np_f32(L.forward())
    assert np.array_equal(a, b)                    # ordered sums: bit-identical from run to run
    if case.get("eps") == 0.5 and not case.get("min_k"):
        mask = to_np(L.mask)[:s.T]
        assert (mask == 0).any() and np.all(a[mask == 0] == 0.0)


@pytest.mark.parametrize("cfg,kw,n,fuse", [("c3", {}, 256, 2), ("c5", dict(eps=0.1), 512, 2), ("c5", dict(eps=0.1), 512, 1)],
                         ids=["c3_separate", "c5_eps0.1_separate", "c5_eps0.1_inside"])
def test_both_aggregation_paths_full_size(cfg, kw, n, fuse):
    s = gi.spec(cfg, fuse_combine=fuse, **kw)
    r = layer_parity(s, sample=n)
    assert r["err_rows"] <= TOL_BF16, (r["err_rows"], r["err"])
    if cfg == "c3":
        assert r["err"] <= TOL_BF16


# ---------------------------------------------------------------- a handful of tokens (a decoding step of a few sequences)

FEW = [
    dict(T=1, d=2048, H=1024, E=32, mode=gi.MODE_THRESHOLD, eps=0.03),
    dict(T=3, d=512, H=256, E=16, mode=gi.MODE_TOPK, K=2),
    dict(T=7, d=320, H=192, E=8, mode=gi.MODE_ALL),                          # ragged column tiles of the down-projection
    dict(T=5, d=4096, H=512, E=32, mode=gi.MODE_THRESHOLD, eps=0.03),
    dict(T=2, d=128, H=64, E=64, mode=gi.MODE_TOPK, K=3),                    # tiles cross several experts
    dict(T=4, d=64, H=6144, E=8, mode=gi.MODE_ALL),                          # wide experts, short reductions
    dict(T=6, d=256, H=128, E=33, mode=gi.MODE_THRESHOLD, eps=0.02, zipf_s=1.1),   # E % 4 != 0: the router's scalar loads
    dict(T=7, d=256, H=128, E=8, mode=gi.MODE_THRESHOLD, eps=0.999),         # nothing selected: zeros
    dict(T=1, d=64, H=64, E=1, mode=gi.MODE_ALL),
    dict(T=7, d=1024, H=2048, E=4, mode=gi.MODE_TOPK, K=1, out_fp32=1),
]


@pytest.mark.parametrize("case", FEW, ids=[str(i) for i in range(len(FEW))])
def test_few_tokens(case):
    s = gi.LayerSpec(f"few{FEW.index(case)}", dtype="bf16", router_gain=3.0, **case)
    r = layer_parity(s)
    assert r["err_rows"] <= TOL_BF16 and r["err"] <= TOL_BF16, (r["err_rows"], r["err"])
    L = r["layer"]
    a = np_f32(L.forward()).copy()
    assert np.array_equal(a, np_f32(L.forward()))               # fixed summation order: bit-identical run to run
    if case.get("eps") == 0.999:
        assert r["A"] == 0 and np.all(a == 0.0)
