"""Parity of the mixture-of-attention-heads layer (Eq. 7-8) with the CPU oracle (GPU required): the GPU decides the
selection on its own scores (checked against the oracle's as for the feed-forward layer), the oracle evaluates Eq. 8
on the GPU's selection.  Shapes follow Table `tab:model_arch` (n_head x d_head = 2 x 64, 4 x 96, 4 x 128 per expert, 8
or 16 experts), with prefill-like batches of several sequences and decode-like batches of one token per sequence."""
import math

import numpy as np
import pytest
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm
from harness import TOL_BF16, check_mask_against_oracle, desc_of, record, rel_err, rel_err_rows, to_dev, to_np

pytestmark = pytest.mark.gpu


def _moa_case(name, T, d, E, n_head, dh, n_seq, L, layout, mode, **sel):
    """layout 'prefill': the T tokens are n_seq sequences of T / n_seq tokens at positions 0, 1, ...; 'decode': one
    new token per sequence (T == n_seq) at seeded positions; 'mixed': seeded sequences and positions; 'full': seeded
    sequences, every token at the cache's last position."""
    H = n_head * dh
    s = gi.LayerSpec(name, T=T, d=d, H=H, E=E, dtype="bf16", mode=mode, router_gain=4.0, **sel)
    x = gi.tokens(s)
    Wr, br = gi.router(s)
    Wq, Wo = gi.experts(s)                                   # [E, d, H], [E, H, d]: same shapes as the expert MLPs' weights
    Kc = gi.normal(s.seed, f"{name}.K", (n_seq, n_head, L, dh), 1.0, "bf16")
    Vc = gi.normal(s.seed, f"{name}.V", (n_seq, n_head, L, dh), 1.0, "bf16")
    u = gi.uniform(s.seed, f"{name}.pos", T)
    if layout == "prefill":
        per = T // n_seq
        seq = (np.arange(T) // per).astype(np.int32)
        pos = (np.arange(T) % per).astype(np.int32)
    elif layout == "decode":
        seq = np.arange(T, dtype=np.int32)
        pos = np.minimum((u * L).astype(np.int32), L - 1)
        pos[0], pos[-1] = L - 1, 0
    else:
        seq = np.minimum((gi.uniform(s.seed, f"{name}.seq", T) * n_seq).astype(np.int32), n_seq - 1)
        pos = np.minimum((u * L).astype(np.int32), L - 1)
        if layout == "full":                                 # every token sees the whole cache
            pos[:] = L - 1
    return s, x, Wr, br, Wq, Wo, Kc, Vc, seq, pos


def _run(s, x, Wr, br, Wq, Wo, Kc, Vc, seq, pos, n_head, scale, sample=None, use_seq=True):
    desc = desc_of(s.replace(out_fp32=1))
    x_d, Wr_d, br_d = to_dev(x), to_dev(Wr), to_dev(br)
    packed = torch.empty(dm.dsmoe_packed_size(desc), dtype=torch.uint8, device="cuda")
    dm.dsmoe_pack_weights(desc, to_dev(Wq), to_dev(Wo), packed)
    ws = torch.empty(dm.dsmoe_workspace_size_packed(desc), dtype=torch.uint8, device="cuda")
    out = torch.empty((s.T, s.d), dtype=torch.float32, device="cuda")
    mask = torch.zeros(s.T, dtype=torch.int64, device="cuda")
    counts = torch.zeros(64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    K_d, V_d, seq_d, pos_d = to_dev(Kc), to_dev(Vc), to_dev(seq) if use_seq else None, to_dev(pos)
    dm.dsmoe_moa_forward(desc, n_head, scale, K_d, V_d, seq_d, pos_d, x_d, Wr_d, br_d, packed, out, mask, counts, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    first = out.cpu().numpy().copy()
    dm.dsmoe_moa_forward(desc, n_head, scale, K_d, V_d, seq_d, pos_d, x_d, Wr_d, br_d, packed, out, mask, counts, ws, status)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    assert np.array_equal(first, got)                        # bit-identical from run to run
    mask_gpu = to_np(mask).view(np.uint64)
    S = oracle.router_scores(x, Wr, br)
    mask_ref, _ = oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
    flips, near = check_mask_against_oracle(s, S, mask_gpu, mask_ref)
    ids = None if sample is None or sample >= s.T else gi.sample_tokens(s, sample)
    ref = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask_gpu, pos, n_head, scale, tok_seq=seq if use_seq else None, token_ids=ids)
    g = got if ids is None else got[ids]
    e, er = rel_err(g, ref), rel_err_rows(g, ref)
    record("moa_parity", name=s.name, T=s.T, d=s.d, E=s.E, n_head=n_head, d_head=s.H // n_head, L=int(Kc.shape[2]),
           n_seq=int(Kc.shape[0]), mode=s.mode, tokens_compared=int(ref.shape[0]), err_global=e, err_per_token=er,
           flips=flips, near_threshold=near, A=int(to_np(counts)[:s.E].sum()))
    return e, er


MOA = [
    # name, T, d, E, n_head, d_head, n_seq, L, layout, mode, selection
    ("moa_1b_prefill", 512, 2048, 16, 2, 64, 4, 128, "prefill", gi.MODE_TOPK, dict(K=6)),
    ("moa_3b_prefill", 384, 3072, 8, 4, 96, 3, 128, "prefill", gi.MODE_TOPK, dict(K=5)),
    ("moa_6b_prefill", 512, 4096, 8, 4, 128, 2, 256, "prefill", gi.MODE_THRESHOLD, dict(eps=0.08)),
    ("moa_6b_decode", 32, 4096, 8, 4, 128, 32, 700, "decode", gi.MODE_THRESHOLD, dict(eps=0.08)),
    ("moa_1b_decode", 5, 2048, 16, 2, 64, 5, 333, "decode", gi.MODE_TOPK, dict(K=3)),
    ("moa_all", 300, 256, 8, 2, 32, 7, 61, "mixed", gi.MODE_ALL, dict()),                       # the dense form the paper runs at inference
    ("moa_one_token", 1, 512, 4, 2, 64, 1, 1, "decode", gi.MODE_ALL, dict()),                   # a single key
    ("moa_empty_rows", 260, 256, 16, 2, 64, 3, 50, "mixed", gi.MODE_THRESHOLD, dict(eps=0.3)),  # tokens that select nothing
    ("moa_wide_head", 200, 512, 4, 1, 256, 2, 90, "mixed", gi.MODE_TOPK, dict(K=2)),
    ("moa_ttk", 513, 256, 8, 4, 32, 4, 140, "mixed", gi.MODE_THRESHOLD_TOPK, dict(eps=0.03)),
    ("moa_many_experts", 70, 256, 40, 2, 64, 2, 50, "mixed", gi.MODE_ALL, dict()),               # 40 rows per token: three row tiles
    ("moa_many_experts_topk", 600, 256, 24, 2, 64, 3, 90, "mixed", gi.MODE_TOPK, dict(K=20)),      # 20 rows per token: two row tiles
    ("moa_full_cache", 300, 1024, 8, 4, 64, 6, 200, "full", gi.MODE_TOPK, dict(K=4)),
    ("moa_full_cache_6b", 64, 4096, 8, 4, 128, 8, 1000, "full", gi.MODE_TOPK, dict(K=5)),
]


@pytest.mark.parametrize("case", MOA, ids=[c[0] for c in MOA])
def test_moa_layer(case):
    name, T, d, E, nh, dh, n_seq, L, layout, mode, sel = case
    s, *rest = _moa_case(name, T, d, E, nh, dh, n_seq, L, layout, mode, **sel)
    e, er = _run(s, *rest, nh, 1.0 / math.sqrt(dh))
    assert er <= TOL_BF16, (e, er)
    # The whole-output form of the bar is asserted where the rows are of one scale.  A token at cache position p
    # averages p + 1 value vectors, so its row is about sqrt((L + 1) / (p + 1)) times larger than that of a token that
    # sees the whole cache: with positions spread over the cache the early tokens' rounding alone exceeds a bar
    # relative to the whole output's RMS (measured: 2.1e-2 to 2.7e-2 there, against 0.8e-2 to 1.3e-2 per token).
    if layout == "full":
        assert e <= TOL_BF16, (e, er)


def test_moa_without_sequence_list_and_with_scale_one():
    s, x, Wr, br, Wq, Wo, Kc, Vc, seq, pos = _moa_case("moa_one_seq", 130, 256, 8, 2, 64, 1, 130, "prefill", gi.MODE_TOPK, K=3)
    e, er = _run(s, x, Wr, br, Wq, Wo, Kc, Vc, seq, pos, 2, 1.0, use_seq=False)
    assert er <= TOL_BF16, (e, er)


def test_moa_fused_and_separate_aggregation():
    for fuse in (1, 2):
        s, *rest = _moa_case(f"moa_fuse{fuse}", 700, 512, 8, 4, 64, 5, 140, "prefill", gi.MODE_TOPK, K=4, fuse_combine=fuse)
        e, er = _run(s, *rest, 4, 0.125)
        assert er <= TOL_BF16, (fuse, e, er)


def test_moa_paper_6b_shape_on_sampled_tokens():
    """DS-MoE-6B's attention layer (8 experts of 4 heads of 128, model width 4096) on 32 sequences of 256 tokens,
    the sequence length of the paper's input-throughput setting; the oracle evaluates 256 seeded tokens."""
    s, *rest = _moa_case("moa_6b_full", 8192, 4096, 8, 4, 128, 32, 256, "prefill", gi.MODE_TOPK, K=5)
    e, er = _run(s, *rest, 4, 1.0 / math.sqrt(128), sample=256)
    assert er <= TOL_BF16, (e, er)


def test_moa_rejects_what_it_does_not_support():
    desc = dm.make_desc(64, 256, 96, 4, dm.BF16, dm.SELECT_ALL)            # H = 96 is not a multiple of 64
    z = torch.zeros(16, dtype=torch.uint8, device="cuda")
    K = torch.zeros((1, 2, 8, 48), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dm.DsmoeError) as ei:
        dm.dsmoe_moa_forward(desc, 2, 1.0, K, K, None, z, z, z, None, z, z, None, None, z)
    assert ei.value.code in (1, 2)


def test_moa_plain_attention_kernel_on_a_common_head_width(monkeypatch):
    """Head widths 64, 96 and 128 normally take the tensor-core attention kernel; the plain one (other widths) is run on
    such a shape too, through the library's switch for it."""
    monkeypatch.setenv("DSMOE_MOA_PLAIN", "1")
    s, *rest = _moa_case("moa_plain", 200, 512, 8, 2, 64, 3, 77, "mixed", gi.MODE_TOPK, K=3)
    e, er = _run(s, *rest, 2, 0.125)
    assert er <= TOL_BF16, (e, er)
