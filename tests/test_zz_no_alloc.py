"""dsmoe_select_static: the selection entry point for callers that cannot allocate device memory.

Such callers (code under a framework-owned allocator, plugins that receive only their inputs and
outputs) have no workspace to pass, so the library keeps that scratch in a fixed device array.  The
results must be bit-identical to dsmoe_select's.  Two calls in a row with different shapes check
that what the first call leaves in the shared array never leaks into the second.
This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm

pytestmark = pytest.mark.gpu


def _scores(name, T, E):
    raw = gi.normal(11, name, (T, E), 1.5, "f32").astype(np.float64)
    p = np.exp(raw - raw.max(1, keepdims=True))
    return torch.from_numpy((p / p.sum(1, keepdims=True)).astype(np.float32)).cuda()


def _outputs(T, E):
    return (torch.zeros(T, dtype=torch.int64, device="cuda"), torch.zeros(T, dtype=torch.int32, device="cuda"),
            torch.full((E,), -1, dtype=torch.int32, device="cuda"),
            torch.full((E + 1,), -1, dtype=torch.int32, device="cuda"))


def _both(desc, S):
    ws = torch.empty(dm.dsmoe_workspace_size(desc), dtype=torch.uint8, device="cuda")
    ref = _outputs(desc.T, desc.E)
    dm.dsmoe_select(desc, S, *ref, ws)
    got = _outputs(desc.T, desc.E)
    dm.dsmoe_select_static(desc, S, *got)
    torch.cuda.synchronize()
    for a, b in zip(got, ref):
        assert torch.equal(a, b)
    # ... and both against the CPU oracle's selection and grouping of the same scores
    S_np = S.cpu().numpy()
    mask_ref, k_ref = oracle.select(S_np, desc.mode, desc.eps, desc.eps_normalized, desc.K, desc.min_k)
    g = oracle.group(mask_ref, S_np, width=dm.width(desc))
    assert np.array_equal(got[0].cpu().numpy().view(np.uint64), mask_ref)
    assert np.array_equal(got[1].cpu().numpy(), k_ref)
    assert np.array_equal(got[2].cpu().numpy(), g["counts"])
    assert np.array_equal(got[3].cpu().numpy(), g["offsets"])
    return got


def test_static_select_matches_select_on_two_calls_in_a_row():
    d1 = dm.make_desc(4099, 64, 64, 64, dm.BF16, dm.SELECT_THRESHOLD, eps=0.02)
    got1 = _both(d1, _scores("na1", d1.T, d1.E))
    assert int(got1[3][-1].item()) == int(got1[1].sum().item()) > 0
    # smaller second call, other rule: stale counts of the first call sit in the shared array
    d2 = dm.make_desc(77, 64, 64, 5, dm.BF16, dm.SELECT_TOPK, K=2)
    got2 = _both(d2, _scores("na2", d2.T, d2.E))
    assert int(got2[3][-1].item()) == 77 * 2
    # and the first shape once more
    _both(d1, _scores("na3", d1.T, d1.E))


def test_static_select_rejects_sizes_beyond_its_built_in_scratch():
    big = dm.make_desc(70000, 64, 64, 64, dm.BF16, dm.SELECT_ALL)      # ceil(70000/32)*64 > 131072
    S = torch.empty(1, dtype=torch.float32, device="cuda")
    outs = _outputs(1, 64)
    with pytest.raises(dm.DsmoeError) as ei:
        dm.dsmoe_select_static(big, S, *outs)
    assert ei.value.code == 3
    ok = dm.make_desc(65536, 64, 64, 64, dm.BF16, dm.SELECT_ALL)       # exactly at the limit
    S = torch.full((ok.T, ok.E), 1.0 / 64, dtype=torch.float32, device="cuda")
    got = _outputs(ok.T, ok.E)
    dm.dsmoe_select_static(ok, S, *got)
    torch.cuda.synchronize()
    assert torch.all(got[2] == 65536) and int(got[3][-1].item()) == 65536 * 64
