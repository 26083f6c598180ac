"""End-to-end parity of dsmoe_layer_forward against the CPU oracle (GPU required)."""
import numpy as np
import pytest
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm
from harness import TOL_BF16, TOL_F32, Layer, layer_parity, np_f32, to_np

pytestmark = pytest.mark.gpu


def test_c1_tiny_fp32_threshold_layer():
    s = gi.spec("c1")
    r = layer_parity(s)
    assert r["err"] <= TOL_F32
    frac = r["A"] / (s.T * s.E)
    assert 0.30 <= frac <= 0.40                       # the recipe's 35 % active experts


SMALL = [
    dict(T=7, d=64, H=64, E=3, mode=gi.MODE_THRESHOLD, eps=0.2),
    dict(T=129, d=128, H=72, E=33, mode=gi.MODE_TOPK, K=4),
    dict(T=33, d=256, H=136, E=64, mode=gi.MODE_THRESHOLD, eps=0.01, zipf_s=1.1),
    dict(T=200, d=128, H=128, E=8, mode=gi.MODE_ALL),
    dict(T=1, d=64, H=64, E=1, mode=gi.MODE_ALL),
    dict(T=300, d=64, H=64, E=16, mode=gi.MODE_THRESHOLD, eps=0.5),              # most tokens select nothing
    dict(T=300, d=64, H=64, E=16, mode=gi.MODE_THRESHOLD, eps=0.5, min_k=1),
    dict(T=64, d=64, H=64, E=2, mode=gi.MODE_TOPK, K=2, out_fp32=1),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("pack", [False, True], ids=["plain", "packed"])
@pytest.mark.parametrize("case", SMALL, ids=[str(i) for i in range(len(SMALL))])
def test_small_layers(case, pack, dtype):
    if pack and dtype == "f32":
        pytest.skip("packed weights are bf16 only")
    s = gi.LayerSpec(f"small{SMALL.index(case)}", dtype=dtype, router_gain=6.0, **case)
    r = layer_parity(s, pack=pack)
    tol = TOL_F32 if dtype == "f32" else TOL_BF16
    # adversarial shapes mix tokens with very different numbers of experts: the bar is applied per token ...
    assert r["err_rows"] <= tol, (r["err_rows"], r["err"])
    # ... and over the whole output as well, except where most tokens select nothing: their rows of exact zeros
    # pull the whole-output RMS far below that of the rows that carry values (measured there: up to 8e-2)
    if case.get("eps") != 0.5:
        assert r["err"] <= tol, r["err"]
    if case.get("eps") == 0.5 and not case.get("min_k"):
        assert r["zero_tokens"] > 0
        out = np_f32(r["layer"].out)
        mask = to_np(r["layer"].mask)[:s.T]
        assert np.all(out[mask == 0] == 0.0)          # Eq. 1 with an empty selection is the zero vector


@pytest.mark.parametrize("T,E,sel", [
    (16384 + 70, 8, dict(mode=gi.MODE_TOPK, K=2)),            # beyond 512 chunks: the one-block scan kernel between counts and rows
    (16384, 40, dict(mode=gi.MODE_THRESHOLD, eps=0.04)),      # exactly 512 chunks, 64-wide expert words: every block scans itself
    (250, 8, dict(mode=gi.MODE_TOPK, K=3)),                   # up to 8 chunks: every block also counts from the masks
    (257, 24, dict(mode=gi.MODE_THRESHOLD, eps=0.06)),        # 9 chunks, the tensor-core router's counts
], ids=["scan_kernel", "scan_in_block_512", "count_in_block", "router_counts"])
def test_grouping_forms_of_the_fused_layer(T, E, sel):
    """The three ways the fused layer gets from masks to grouped rows (by number of 32-token chunks), each on a ragged
    token count; selection, counts and the layer output against the oracle on a sample that reaches every expert."""
    s = gi.LayerSpec(f"group{T}", T=T, d=64, H=64, E=E, dtype="bf16", router_gain=5.0, **sel)
    r = layer_parity(s, sample=768)
    assert r["err_rows"] <= TOL_BF16, (r["err_rows"], r["err"])
    assert r["err"] <= TOL_BF16, r["err"]
    L = r["layer"]
    # the tail of the batch is where a wrong prefix over the chunks shows: compare the last tokens one by one
    ids = np.arange(s.T - 40, s.T)
    S = L.oracle_scores()
    mask = to_np(L.mask)[:s.T].view(np.uint64)
    ref = oracle.layer(L.x, L.W1, L.W2, S, mask, token_ids=ids)
    got = np_f32(L.forward(out_fp32=True))[ids]
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    assert float(np.abs(got - ref).max()) <= TOL_BF16 * rms


def test_all_tokens_to_one_expert_and_empty_experts():
    s = gi.LayerSpec("onehot", T=150, d=64, H=64, E=8, dtype="bf16", mode=gi.MODE_TOPK, K=1)
    L = Layer(s)
    br = np.zeros(s.E, np.float32)
    br[5] = 50.0
    L.br, L.br_d = br, torch.from_numpy(br).cuda()
    out = np_f32(L.forward())
    counts = to_np(L.counts)[:s.E]
    assert counts.tolist() == [0, 0, 0, 0, 0, 150, 0, 0]
    S = L.oracle_scores()
    mask, _ = L.oracle_select(S)
    ref = oracle.layer(L.x, L.W1, L.W2, S, mask)
    from harness import rel_err
    assert rel_err(out, ref) <= TOL_BF16


def test_t0_is_a_noop():
    desc = dm.make_desc(0, 64, 64, 4, dm.BF16)
    dm.dsmoe_layer_forward(desc, None, None, None, None, None, None, None, None, None, None)


def test_selection_is_reproducible_run_to_run():
    s = gi.LayerSpec("repro", T=777, d=128, H=64, E=32, dtype="bf16", mode=gi.MODE_THRESHOLD, eps=0.03,
                     router_gain=4.0)
    L = Layer(s)
    a = np_f32(L.forward()).copy()
    m1 = to_np(L.mask).copy()
    b = np_f32(L.forward())
    assert np.array_equal(m1, to_np(L.mask)) and np.array_equal(a, b)


# ---------------------------------------------------------------- the five benchmark workloads

@pytest.mark.parametrize("T", [1, 8, 32, 128])
def test_c2_decode_shaped_layer(T):
    s = gi.spec("c2", T=T)
    r = layer_parity(s)
    assert r["err"] <= TOL_BF16, r["err"]
    if T >= 32:
        assert 0.25 <= r["A"] / (s.T * s.E) <= 0.45     # the recipe's 30-40 % active experts


def test_c3_prefill_shaped_layer_topk():
    s = gi.spec("c3")
    r = layer_parity(s, sample=1024)
    assert r["A"] == s.T * s.K                           # top-K: exactly K experts per token
    assert r["err"] <= TOL_BF16, r["err"]


def test_c4_dense_forward_all_experts():
    s = gi.spec("c4")
    r = layer_parity(s, sample=1024)
    assert r["A"] == s.T * s.E
    assert r["err"] <= TOL_BF16, r["err"]


@pytest.mark.parametrize("eps", [0.0, 0.01, 0.05, 0.1, 0.2])
def test_c5_skewed_router_threshold_sweep(eps):
    s = gi.spec("c5", eps=eps)
    r = layer_parity(s, sample=256 if eps == 0.0 else 1024)
    if eps == 0.0:
        assert r["A"] == s.T * s.E                       # no score underflows to 0 in this recipe
    if eps >= 0.1:
        assert r["empty_experts"] > 0 or r["zero_tokens"] > 0
    # rows differ wildly in scale here (1 to 64 experts per token): the bar is applied per token; the bar over the
    # whole output holds too while few tokens select nothing (eps = 0.2: 28 % of the rows are exact zeros)
    assert r["err_rows"] <= TOL_BF16, (r["err_rows"], r["err"])
    if eps < 0.1:
        assert r["err"] <= TOL_BF16, r["err"]


# ---------------------------------------------------------------- decode path corner cases
# The decode kernel streams only the experts that some token selected and cuts that list evenly over
# the CTAs: few, no, skewed and all experts selected.

@pytest.mark.parametrize("case", [
    dict(T=24, E=32, mode=gi.MODE_TOPK, K=1),                       # at most 24 of 32 experts selected
    dict(T=16, E=16, mode=gi.MODE_THRESHOLD, eps=0.4),              # a few experts, many tokens with none
    dict(T=40, E=8, mode=gi.MODE_THRESHOLD, eps=0.999),             # no expert at all: the output is zero
    dict(T=128, E=64, mode=gi.MODE_TOPK, K=2, zipf_s=1.1),          # skewed: popular experts only
    dict(T=17, E=4, mode=gi.MODE_ALL),                              # every expert (the assumption holds)
    # wide experts: several up-projection tiles per CTA, short reductions, so streaming under "every expert
    # selected" runs far ahead of the router before it is confirmed (all) or has to start over (topk1)
    dict(T=20, E=8, mode=gi.MODE_ALL, d=128, H=6144),
    dict(T=20, E=16, mode=gi.MODE_TOPK, K=1, d=128, H=3072),
    dict(T=32, E=16, mode=gi.MODE_TOPK, K=1, d=2048, H=128),         # ... and long reductions: it starts over mid-tile
    # nearly every expert selected: the up-projection started under "every expert" stands, the unselected experts'
    # tiles are gated to zero and the down-projection runs over the selected ones only (15 and 14 of 16); with 12 of
    # 16 it starts over
    dict(T=12, E=16, mode=gi.MODE_TOPK, K=3),
    dict(T=9, E=16, mode=gi.MODE_TOPK, K=3),
    dict(T=9, E=16, mode=gi.MODE_TOPK, K=2),
    dict(T=12, E=16, mode=gi.MODE_TOPK, K=3, d=128, H=3072),
], ids=["topk1", "few", "none", "skew", "all", "wide_all", "wide_topk1", "deep_topk1", "near15", "near14", "far12",
        "wide_near15"])
def test_decode_path_when_some_experts_are_unselected(case):
    kw = dict(d=512, H=256)
    kw.update(case)
    s = gi.LayerSpec("dec_" + str(case["T"]), dtype="bf16", router_gain=8.0, **kw)
    r = layer_parity(s)
    assert r["err_rows"] <= TOL_BF16, (r["err_rows"], r["err"])
    assert r["err"] <= TOL_BF16, r["err"]
    if case.get("eps") == 0.999:
        assert r["A"] == 0 and np.all(np_f32(r["layer"].out) == 0.0)
    if case["mode"] == gi.MODE_TOPK and case["K"] == 1:
        assert r["empty_experts"] >= (8 if case["E"] == 32 else 1)


# ---------------------------------------------------------------- Threshold-TopK ("Expert Sampling Strategy" paragraph)

@pytest.mark.parametrize("case", [
    dict(T=40, d=128, H=128, E=8, eps=0.06),                  # few tokens: not the one-launch decode kernel (K needs the batch)
    dict(T=300, d=128, H=64, E=16, eps=0.03),
    dict(T=1000, d=256, H=128, E=32, eps=0.7, eps_normalized=1, zipf_s=1.1),
    dict(T=513, d=64, H=72, E=5, eps=0.16),                   # plain fp32-FMA path (H % 64 != 0)
], ids=["t40", "t300", "t1000_skew", "plain"])
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_threshold_topk_layer(case, dtype):
    s = gi.LayerSpec("tt_" + str(case["T"]), dtype=dtype, mode=gi.MODE_THRESHOLD_TOPK, router_gain=4.0, **case)
    r = layer_parity(s)
    k = np_popcounts(r["layer"].mask, s.T)
    assert len(set(k.tolist())) == 1 and 1 <= int(k[0]) <= s.E        # every token got the same K
    assert r["A"] == s.T * int(k[0])
    tol = TOL_BF16 if dtype == "bf16" else TOL_F32
    assert r["err_rows"] <= tol and r["err"] <= tol, (r["err_rows"], r["err"])


def np_popcounts(mask_t, T):
    m = mask_t.cpu().numpy()[:T].view(np.uint64)
    return np.array([bin(int(v)).count("1") for v in m])


# ---------------------------------------------------------------- the paper's own layer shapes (Table tab:model_arch)
# DS-MoE-1B / 3B / 6B: 32 experts of width 256 / 384 / 512 at model width 2048 / 3072 / 4096 -- narrower experts
# than the benchmark configurations, so other tile widths, ring geometries and partitions.

PAPER_SHAPES = [("1b", 2048, 256), ("3b", 3072, 384), ("6b", 4096, 512)]


@pytest.mark.parametrize("name,d,H", PAPER_SHAPES, ids=[p[0] for p in PAPER_SHAPES])
@pytest.mark.parametrize("T", [1, 16, 48])
def test_paper_shaped_decode(name, d, H, T):
    s = gi.LayerSpec(f"paper_{name}_t{T}", T=T, d=d, H=H, E=32, dtype="bf16", mode=gi.MODE_THRESHOLD, eps=0.03,
                     router_gain=2.0)
    r = layer_parity(s)
    assert r["err_rows"] <= TOL_BF16 and r["err"] <= TOL_BF16, (r["err_rows"], r["err"])


@pytest.mark.parametrize("name,d,H", PAPER_SHAPES, ids=[p[0] for p in PAPER_SHAPES])
@pytest.mark.parametrize("K", [4, 6])
def test_paper_shaped_prefill_topk(name, d, H, K):
    s = gi.LayerSpec(f"paper_{name}_k{K}", T=2048, d=d, H=H, E=32, dtype="bf16", mode=gi.MODE_TOPK, K=K)
    r = layer_parity(s, sample=256)
    assert r["A"] == 2048 * K
    assert r["err_rows"] <= TOL_BF16 and r["err"] <= TOL_BF16, (r["err_rows"], r["err"])


# ---------------------------------------------------------------- the scaled models of the paper's speed test (Table tab:scaled)
# DS-MoE-10B / 14B / 19B: 32 experts of width 640 / 768 / 896 at model width 5120 / 6144 / 7168, top-K 4.

SCALED_SHAPES = [("10b", 5120, 640), ("14b", 6144, 768), ("19b", 7168, 896)]


@pytest.mark.parametrize("name,d,H", SCALED_SHAPES, ids=[p[0] for p in SCALED_SHAPES])
@pytest.mark.parametrize("T", [1, 32, 1024])
def test_scaled_model_shapes(name, d, H, T):
    s = gi.LayerSpec(f"scaled_{name}_t{T}", T=T, d=d, H=H, E=32, dtype="bf16", mode=gi.MODE_TOPK, K=4, router_gain=2.0)
    r = layer_parity(s, sample=64 if T > 64 else None)
    assert r["A"] == T * 4
    assert r["err_rows"] <= TOL_BF16 and r["err"] <= TOL_BF16, (r["err_rows"], r["err"])


# ---------------------------------------------------------------- a stack of layers: layer i's output is layer i + 1's input
# (output-token throughput as the "GPU Inference Analysis" section measures it).  Every layer of the stack is checked
# against the oracle on the very activations the previous layer produced on the GPU.

@pytest.mark.parametrize("T", [1, 8, 40, 300])
def test_stack_of_layers_feeding_one_another(T):
    n_layers = 6
    s = gi.LayerSpec(f"stack_t{T}", T=T, d=512, H=256, E=16, dtype="bf16", mode=gi.MODE_THRESHOLD, eps=0.04,
                     router_gain=2.0, w2_gain=32.0)
    x = gi.tokens(s)
    x_d = None
    rms = []
    for layer in range(n_layers):
        L = Layer(s, layer=layer)
        if x_d is not None:
            L.x_d, L.x = x_d, to_np(x_d)                      # the previous layer's bf16 output, bit for bit
        out32 = L.forward(out_fp32=True).cpu().numpy()
        out16 = L.forward(out_fp32=False)
        assert torch.equal(out16, torch.from_numpy(out32).cuda().to(torch.bfloat16))
        mask_gpu = to_np(L.mask)[:T].view(np.uint64)
        S = oracle.router_scores(L.x, L.Wr, L.br)
        mask_ref, _ = oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
        from harness import check_mask_against_oracle, rel_err_rows
        check_mask_against_oracle(s, S, mask_gpu, mask_ref)
        ref = oracle.layer(L.x, L.W1, L.W2, S, mask_gpu)
        assert rel_err_rows(out32, ref) <= TOL_BF16
        rms.append(float(np.sqrt(np.mean(ref ** 2))))
        x_d = out16.clone()
    from harness import record
    record("layer_stack", T=T, layers=n_layers, rms_per_layer=rms)
    assert all(np.isfinite(rms)) and rms[-1] > 0.0


# ---------------------------------------------------------------- host-buffer entry points

@pytest.mark.parametrize("T", [32, 300])
def test_host_buffer_calls_match_the_device_call(T):
    """dsmoe_layer_forward_host and its un-waited form give, in host memory, exactly the device call's output;
    two un-waited calls on two streams with their own buffers do not disturb one another."""
    s = gi.LayerSpec("host", T=T, d=256, H=128, E=16, dtype="bf16", mode=gi.MODE_THRESHOLD, eps=0.05, router_gain=4.0)
    L = Layer(s)
    ref = L.forward().cpu()
    x_host = L.x_d.cpu().pin_memory()
    out_host = torch.zeros((s.T, s.d), dtype=torch.bfloat16).pin_memory()
    x_dev = torch.zeros_like(L.x_d)
    out_dev = torch.zeros_like(L.out)
    dm.dsmoe_layer_forward_host(L.desc, x_host, x_dev, L.Wr_d, L.br_d, L.W1_d, L.W2_d, L.packed, out_dev, out_host,
                                L.ws, L.dev_status)
    assert int(L.dev_status.item()) == 0
    assert torch.equal(out_host, ref)              # no synchronize here: the call itself waited
    # two calls in flight at once: the second one's input is the first one's tokens in reverse order
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    x2_host = x_host.flip(0).contiguous().pin_memory()
    outs = [torch.zeros_like(out_host).pin_memory() for _ in range(2)]
    bufs = [(torch.zeros_like(L.x_d), torch.zeros_like(L.out), torch.empty_like(L.ws), torch.zeros_like(L.dev_status))
            for _ in range(2)]
    torch.cuda.synchronize()
    for i, xh in enumerate((x_host, x2_host)):
        xd, od, ws, st = bufs[i]
        dm.dsmoe_layer_forward_host_async(L.desc, xh, xd, L.Wr_d, L.br_d, L.W1_d, L.W2_d, L.packed, od, outs[i], ws, st,
                                          stream=streams[i])
    for st in streams:
        st.synchronize()
    assert all(int(b[3].item()) == 0 for b in bufs)
    assert torch.equal(outs[0], ref)
    assert torch.equal(outs[1], ref.flip(0))       # a token's output does not depend on its place in the batch
