"""Pins for the CPU oracle: closed forms, invariants, library special cases, brute force.

The paper prints no numeric example of the layer, so every pin here is something the
paper's equations or plain mathematics fix independently of the oracle's own code.
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.special import erf, softmax

import dsmoe_inputs as gi
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(name, shape, scale=1.0, dtype="f32", seed=7):
    return gi.normal(seed, name, shape, scale, dtype)


def _np_gelu(v):
    return 0.5 * v * (1.0 + erf(v / math.sqrt(2.0)))


def _np_expert(xrow, W1e, W2e):
    return _np_gelu(xrow @ W1e) @ W2e


# ---------------------------------------------------------------- scores (Eq. 1)

def test_scores_match_library_softmax_of_numpy_logits():
    T, d, E = 37, 48, 11
    x, Wr, br = _rand("x", (T, d)), _rand("Wr", (d, E), 0.3), _rand("br", (E,), 0.5)
    S = oracle.router_scores(x, Wr, br)
    ref = softmax(x.astype(np.float64) @ Wr.astype(np.float64) + br.astype(np.float64), axis=1)
    assert S.dtype == np.float32
    np.testing.assert_allclose(S, ref, rtol=1e-7, atol=0)       # one fp32 rounding of the exact value
    assert np.array_equal(S, ref.astype(np.float32))


def test_scores_sum_to_one_and_shift_invariance():
    T, d, E = 64, 32, 32
    x, Wr, br = _rand("x2", (T, d)), _rand("Wr2", (d, E), 0.5), _rand("br2", (E,))
    S = oracle.router_scores(x, Wr, br)
    assert np.all(np.abs(S.astype(np.float64).sum(1) - 1.0) < 4 * E * np.finfo(np.float32).eps)
    S2 = oracle.router_scores(x, Wr, br + np.float32(3.0))
    np.testing.assert_allclose(S2, S, rtol=2e-6)


def test_scores_uniform_when_router_is_zero():
    for E in (1, 2, 3, 8, 33, 64):
        x = _rand("x3", (5, 16))
        S = oracle.router_scores(x, np.zeros((16, E), np.float32), np.zeros(E, np.float32))
        assert np.all(S == np.float32(1.0 / E))


def test_scores_one_hot_for_large_gain():
    T, d, E = 9, 8, 6
    hot = np.arange(T) % E
    br = np.zeros(E, np.float32)
    # token t sees logit 200 on expert hot[t] through a per-token one-hot feature
    x = np.zeros((T, E), np.float32)
    x[np.arange(T), hot] = 1.0
    Wr = (200.0 * np.eye(E)).astype(np.float32)
    S = oracle.router_scores(x, Wr, br)
    expect = np.zeros((T, E), np.float32)
    expect[np.arange(T), hot] = 1.0
    assert np.array_equal(S, expect)


def test_scores_read_bf16_bits_exactly():
    T, d, E = 6, 24, 5
    xb = _rand("xb", (T, d), 1.0, "bf16")
    Wr = _rand("Wrb", (d, E), 0.2)
    S_bits = oracle.router_scores(xb, Wr)
    S_vals = oracle.router_scores(gi.bf16_to_f32(xb), Wr)
    assert np.array_equal(S_bits, S_vals)


# ---------------------------------------------------------------- selection

def _scores(T, E, name, gain=2.0):
    x, Wr = _rand(name + "x", (T, 16)), _rand(name + "W", (16, E), gain / 4)
    return oracle.router_scores(x, Wr)


def test_threshold_is_strict_and_matches_definition():
    S = np.array([[0.5, 0.25, 0.25], [0.1, 0.1, 0.8]], np.float32)
    m, k = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.25)
    assert m.tolist() == [0b001, 0b100] and k.tolist() == [1, 1]       # equality does not pass
    m, k = oracle.select(S, oracle.MODE_THRESHOLD, eps=np.nextafter(np.float32(0.25), np.float32(0)))
    assert m.tolist() == [0b111, 0b100]
    S = _scores(50, 12, "thr")
    for eps in (0.0, 0.03, 0.1, 0.4):
        m, k = oracle.select(S, oracle.MODE_THRESHOLD, eps=eps)
        brute = [(S[t] > np.float32(eps)) for t in range(50)]
        for t in range(50):
            assert [(int(m[t]) >> e) & 1 for e in range(12)] == brute[t].astype(int).tolist()
            assert k[t] == brute[t].sum()


def test_threshold_normalised_probability_footnote():
    # normalised probability = S * N; with N a power of two the product is exact, so the
    # rule must coincide with the raw rule at eps / N.
    for E in (8, 32, 64):
        S = _scores(40, E, f"norm{E}")
        for eps in (0.3, 0.48, 0.9, 1.5):
            m1, _ = oracle.select(S, oracle.MODE_THRESHOLD, eps=eps, eps_normalized=1)
            m2, _ = oracle.select(S, oracle.MODE_THRESHOLD, eps=eps / E, eps_normalized=0)
            assert np.array_equal(m1, m2)
    # general N: fp32 product compared with eps
    S = _scores(40, 7, "norm7")
    m, _ = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.48, eps_normalized=1)
    for t in range(40):
        bits = [(int(m[t]) >> e) & 1 for e in range(7)]
        assert bits == [int(np.float32(S[t, e] * np.float32(7)) > np.float32(0.48)) for e in range(7)]
    # eps < 1 on the normalised scale always keeps the argmax (max S >= 1/N)
    assert np.all(oracle.select(S, oracle.MODE_THRESHOLD, eps=0.99, eps_normalized=1)[1] >= 1)


def test_threshold_monotone_in_eps():
    S = _scores(64, 16, "mono")
    prev = None
    for eps in (0.0, 0.01, 0.05, 0.1, 0.2, 0.5):
        m, _ = oracle.select(S, oracle.MODE_THRESHOLD, eps=eps)
        if prev is not None:
            assert np.all((m & ~prev) == 0)        # mask(eps2) subset of mask(eps1)
        prev = m


def test_threshold_equals_topk_with_adaptive_k():
    # "K ... adaptively, depending on how many experts have scores above a threshold"
    S = _scores(64, 16, "adapt")
    m_thr, k_t = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.06)
    assert len(set(k_t.tolist())) > 2                              # K really varies per token
    for t in range(64):
        assert len(np.unique(S[t])) == 16                          # no ties in this draw
        m_top, _ = oracle.select(S[t:t + 1], oracle.MODE_TOPK, K=int(k_t[t]))
        assert m_top[0] == m_thr[t]


def test_topk_brute_force_subsets_and_nesting():
    for E in (1, 2, 3, 5, 8):
        S = _scores(12, E, f"bf{E}")
        prev = np.zeros(12, np.uint64)
        for K in range(0, E + 1):
            m, k = oracle.select(S, oracle.MODE_TOPK, K=K)
            assert np.all(k == K)
            assert np.all((prev & ~m) == 0)                        # mask_K subset of mask_{K+1}
            prev = m
            for t in range(12):
                best = max(itertools.combinations(range(E), K),
                           key=lambda c: sum(float(S[t, e]) for e in c))
                assert int(m[t]) == sum(1 << e for e in best)
        m, _ = oracle.select(S, oracle.MODE_TOPK, K=E + 3)
        assert np.all(m == np.uint64((1 << E) - 1))


def test_topk_ties_go_to_lower_index_and_all_mode():
    S = np.array([[0.2, 0.3, 0.3, 0.2], [0.25, 0.25, 0.25, 0.25]], np.float32)
    assert oracle.select(S, oracle.MODE_TOPK, K=1)[0].tolist() == [0b0010, 0b0001]
    assert oracle.select(S, oracle.MODE_TOPK, K=3)[0].tolist() == [0b0111, 0b0111]
    m, k = oracle.select(S, oracle.MODE_ALL)
    assert m.tolist() == [0b1111, 0b1111] and k.tolist() == [4, 4]
    S64 = np.full((2, 64), 1 / 64, np.float32)
    m, k = oracle.select(S64, oracle.MODE_ALL)
    assert np.all(m == np.uint64(2**64 - 1)) and np.all(k == 64)


def test_min_k_keeps_argmax_only_when_nothing_selected():
    S = np.array([[0.3, 0.4, 0.3], [0.1, 0.1, 0.8], [0.4, 0.4, 0.2]], np.float32)
    m0, k0 = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.5, min_k=0)
    m1, k1 = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.5, min_k=1)
    assert m0.tolist() == [0, 0b100, 0] and k0.tolist() == [0, 1, 0]
    assert m1.tolist() == [0b010, 0b100, 0b001] and k1.tolist() == [1, 1, 1]


# ---------------------------------------------------------------- grouping

def test_group_handworked_example():
    # 4 tokens, 3 experts; token -> experts: 0:{0,2} 1:{1} 2:{} 3:{0,1,2}
    mask = np.array([0b101, 0b010, 0b000, 0b111], np.uint64)
    S = (np.arange(12, dtype=np.float32).reshape(4, 3) + 1) / 100
    g = oracle.group(mask, S)
    assert g["counts"].tolist() == [2, 2, 2]
    assert g["offsets"].tolist() == [0, 2, 4, 6]
    assert g["row_token"].tolist() == [0, 3, 1, 3, 0, 3]
    assert g["row_expert"].tolist() == [0, 0, 1, 1, 2, 2]
    np.testing.assert_array_equal(g["row_gate"], np.float32([0.01, 0.10, 0.05, 0.11, 0.03, 0.12]))
    assert g["token_rows"].tolist() == [[0, 4, -1], [2, -1, -1], [-1, -1, -1], [1, 3, 5]]


def test_group_invariants_on_random_masks():
    T, E = 129, 33
    S = _scores(T, E, "grp")
    mask, k_t = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.03)
    g = oracle.group(mask, S)
    A = int(k_t.sum())
    assert g["A"] == A == int(g["counts"].sum()) == int(g["offsets"][E])
    assert np.all(np.diff(g["offsets"]) == g["counts"])
    seen = set()
    for e in range(E):
        seg = g["row_token"][g["offsets"][e]:g["offsets"][e + 1]]
        assert np.all(np.diff(seg) > 0)                            # token-ascending inside a segment
        for t in seg:
            assert (int(mask[t]) >> e) & 1
            seen.add((int(t), e))
    assert len(seen) == A                                          # each assignment exactly once
    for t in range(T):
        rows = g["token_rows"][t]
        rows = rows[rows >= 0]
        assert len(rows) == k_t[t]
        assert np.all(g["row_token"][rows] == t)
        assert np.all(np.diff(g["row_expert"][rows]) > 0)          # expert-ascending inside a token
        np.testing.assert_array_equal(g["row_gate"][rows], S[t, g["row_expert"][rows]])


def test_permute_then_unpermute_is_identity():
    # one expert per token, gate 1: gathering rows by row_token then combining returns x
    T, E, d = 40, 5, 12
    x = _rand("pid", (T, d))
    choice = (np.arange(T) * 7) % E
    mask = (np.uint64(1) << choice.astype(np.uint64)).astype(np.uint64)
    g = oracle.group(mask, np.ones((T, E), np.float32))
    xp = x[g["row_token"]]
    back = oracle.combine(xp, g["row_gate"], g["token_rows"])
    assert np.array_equal(back, x.astype(np.float64))


# ---------------------------------------------------------------- layer output (Eq. 1)

def test_gelu_table_values_through_a_scalar_layer():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "gelu_values.txt")) if l[0] not in "#\n"]
    one = np.ones((1, 1, 1), np.float32)
    for xs, phis in rows:
        xv, phi = float(xs), float(phis)
        O = oracle.layer(np.array([[xv]], np.float32), one, one, np.ones((1, 1), np.float32),
                         np.ones(1, np.uint64))
        assert abs(O[0, 0] - xv * phi) < 2e-9


def test_layer_brute_force_python_loops():
    T, d, H, E = 3, 3, 2, 2
    x, W1, W2 = _rand("bx", (T, d)), _rand("bW1", (E, d, H), 0.7), _rand("bW2", (E, H, d), 0.7)
    S = np.array([[0.25, 0.75], [0.5, 0.5], [0.9, 0.1]], np.float32)
    mask = np.array([0b10, 0b11, 0b01], np.uint64)
    O = oracle.layer(x, W1, W2, S, mask)
    for t in range(T):
        for c in range(d):
            acc = 0.0
            for e in range(E):
                if not (int(mask[t]) >> e) & 1:
                    continue
                y = 0.0
                for j in range(H):
                    pre = sum(float(x[t, k]) * float(W1[e, k, j]) for k in range(d))
                    act = 0.5 * pre * (1.0 + math.erf(pre / math.sqrt(2.0)))
                    y += act * float(W2[e, j, c])
                acc += float(S[t, e]) * y
            assert abs(O[t, c] - acc) < 1e-14


def test_select_all_equals_dense_training_forward():
    # threshold 0 / K = E / ALL reproduce the dense all-expert weighted sum of Eq. 3's forward
    T, d, H, E = 10, 24, 16, 6
    x, W1, W2 = _rand("dx", (T, d)), _rand("dW1", (E, d, H), 0.2), _rand("dW2", (E, H, d), 0.2)
    S = oracle.router_scores(x, _rand("dWr", (d, E), 0.3))
    dense = np.zeros((T, d))
    x64, W164, W264 = x.astype(np.float64), W1.astype(np.float64), W2.astype(np.float64)
    for e in range(E):
        dense += S[:, e:e + 1].astype(np.float64) * (_np_gelu(x64 @ W164[e]) @ W264[e])
    for mode, kw in ((oracle.MODE_ALL, {}), (oracle.MODE_TOPK, dict(K=E)),
                     (oracle.MODE_THRESHOLD, dict(eps=0.0))):
        mask, k_t = oracle.select(S, mode, **kw)
        assert np.all(k_t == E)
        np.testing.assert_allclose(oracle.layer(x, W1, W2, S, mask), dense, rtol=1e-12, atol=1e-15)


def test_one_hot_router_reproduces_a_single_expert():
    T, d, H, E = 8, 16, 12, 4
    x, W1, W2 = _rand("ox", (T, d)), _rand("oW1", (E, d, H), 0.3), _rand("oW2", (E, H, d), 0.3)
    hot = np.arange(T) % E
    S = np.zeros((T, E), np.float32)
    S[np.arange(T), hot] = 1.0
    mask, _ = oracle.select(S, oracle.MODE_TOPK, K=1)
    O = oracle.layer(x, W1, W2, S, mask)
    for t in range(T):
        ref = _np_expert(x[t].astype(np.float64), W1[hot[t]].astype(np.float64),
                         W2[hot[t]].astype(np.float64))
        np.testing.assert_allclose(O[t], ref, rtol=1e-12, atol=1e-15)


def test_uniform_router_is_scaled_dense_ffn_of_concatenated_experts():
    # Table tab:model_arch: N_ffd * D_ffd(DS-MoE) = D_ffd(dense); checked on the table, then on
    # a scaled-down layer against a two-matmul dense FFN.
    rows = {l.split()[0]: [int(v) for v in l.split()[1:]]
            for l in open(os.path.join(GOLDEN, "model_arch_table.txt")) if l[0] not in "#\n"}
    for size in ("1B", "3B", "6B"):
        demb, n, dffd = rows[f"DS-MoE-{size}"]
        assert rows[f"Dense-{size}"] == [demb, 1, n * dffd]
    T, d, H, E = 12, 32, 8, 4
    x, W1, W2 = _rand("ux", (T, d)), _rand("uW1", (E, d, H), 0.3), _rand("uW2", (E, H, d), 0.3)
    S = oracle.router_scores(x, np.zeros((d, E), np.float32))
    mask, _ = oracle.select(S, oracle.MODE_ALL)
    W1cat = np.concatenate([W1[e] for e in range(E)], axis=1).astype(np.float64)   # [d, E*H]
    W2cat = np.concatenate([W2[e] for e in range(E)], axis=0).astype(np.float64)   # [E*H, d]
    ref = (1.0 / E) * (_np_gelu(x.astype(np.float64) @ W1cat) @ W2cat)
    np.testing.assert_allclose(oracle.layer(x, W1, W2, S, mask), ref, rtol=1e-12, atol=1e-15)


def test_layer_is_linear_in_w2_and_in_the_gate_and_tokens_are_independent():
    T, d, H, E = 9, 16, 8, 5
    x, W1 = _rand("lx", (T, d)), _rand("lW1", (E, d, H), 0.3)
    W2a, W2b = _rand("lW2a", (E, H, d), 0.3), _rand("lW2b", (E, H, d), 0.3)
    S = oracle.router_scores(x, _rand("lWr", (d, E), 0.5))
    mask, _ = oracle.select(S, oracle.MODE_TOPK, K=2)
    Oa, Ob = oracle.layer(x, W1, W2a, S, mask), oracle.layer(x, W1, W2b, S, mask)
    Osum = oracle.layer(x, W1, (W2a.astype(np.float64) + W2b).astype(np.float32), S, mask)
    np.testing.assert_allclose(Osum, Oa + Ob, rtol=1e-5, atol=1e-7)     # fp32 rounding of W2a+W2b
    O2 = oracle.layer(x, W1, W2a, (S * np.float32(0.5)), mask)
    np.testing.assert_allclose(O2, 0.5 * Oa, rtol=1e-12)
    perm = gi.permutation(3, "perm", T)
    Op = oracle.layer(x[perm], W1, W2a, S[perm], mask[perm])
    assert np.array_equal(Op, Oa[perm])
    ids = np.array([7, 2, 2, 5])
    assert np.array_equal(oracle.layer(x, W1, W2a, S, mask, token_ids=ids), Oa[ids])


def test_zero_selected_experts_gives_zero_output():
    T, d, H, E = 4, 8, 4, 3
    x, W1, W2 = _rand("zx", (T, d)), _rand("zW1", (E, d, H)), _rand("zW2", (E, H, d))
    S = np.full((T, E), 1 / 3, np.float32)
    mask, k_t = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.5)
    assert np.all(k_t == 0)
    assert np.all(oracle.layer(x, W1, W2, S, mask) == 0.0)


def test_stage_functions_agree_with_independent_numpy():
    T, d, H, E = 16, 24, 12, 4
    xb = _rand("sx", (T, d), 1.0, "bf16")
    W1b, W2b = _rand("sW1", (E, d, H), 0.2, "bf16"), _rand("sW2", (E, H, d), 0.2, "bf16")
    x, W1, W2 = (gi.bf16_to_f32(a).astype(np.float64) for a in (xb, W1b, W2b))
    S = oracle.router_scores(xb, _rand("sWr", (d, E), 0.4))
    mask, _ = oracle.select(S, oracle.MODE_TOPK, K=2)
    g = oracle.group(mask, S)
    xp = xb[g["row_token"]]
    yp = oracle.expert_rows(xp, W1b, W2b, g["row_expert"])
    for r in range(g["A"]):
        e = g["row_expert"][r]
        np.testing.assert_allclose(yp[r], _np_expert(x[g["row_token"][r]], W1[e], W2[e]),
                                   rtol=1e-12, atol=1e-15)
    out = oracle.combine(yp.astype(np.float32), g["row_gate"], g["token_rows"])
    ref = np.zeros((T, d))
    for r in range(g["A"]):
        ref[g["row_token"][r]] += float(g["row_gate"][r]) * yp[r].astype(np.float32).astype(np.float64)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-18)
    np.testing.assert_allclose(oracle.layer(xb, W1b, W2b, S, mask), out, rtol=1e-5, atol=1e-7)


# ---------------------------------------------------------------- Threshold-TopK ("Expert Sampling Strategy" paragraph)

def _bits(*experts):
    m = 0
    for e in experts:
        m |= 1 << e
    return m


def test_threshold_topk_worked_example_typed_by_hand():
    # 4 tokens x 4 experts.  Raw threshold 0.2 activates 4, 1, 2 and 2 experts: 9 in all, 2.25 per token on
    # average, so K = 2 and every token keeps its two highest scores (ties go to the lower index).
    S = np.array([[0.30, 0.25, 0.24, 0.21],
                  [0.70, 0.10, 0.10, 0.10],
                  [0.40, 0.40, 0.10, 0.10],
                  [0.15, 0.35, 0.15, 0.35]], dtype=np.float32)
    thr_mask, thr_k = oracle.select(S, oracle.MODE_THRESHOLD, eps=0.2)
    assert list(thr_k) == [4, 1, 2, 2]
    mask, k_t = oracle.select(S, oracle.MODE_THRESHOLD_TOPK, eps=0.2)
    assert list(k_t) == [2, 2, 2, 2]
    assert [int(m) for m in mask] == [_bits(0, 1), _bits(0, 1), _bits(0, 1), _bits(1, 3)]


def test_threshold_topk_rounds_the_average_half_up_and_stays_within_1_and_E():
    # counts (1, 2): average 1.5 -> K = 2;  counts (1, 1, 2): 4/3 -> K = 1
    S2 = np.array([[0.7, 0.2, 0.1], [0.45, 0.45, 0.10]], dtype=np.float32)
    _, k = oracle.select(S2, oracle.MODE_THRESHOLD_TOPK, eps=0.3)
    assert list(k) == [2, 2]
    S3 = np.array([[0.7, 0.2, 0.1], [0.6, 0.25, 0.15], [0.45, 0.45, 0.10]], dtype=np.float32)
    m, k = oracle.select(S3, oracle.MODE_THRESHOLD_TOPK, eps=0.3)
    assert list(k) == [1, 1, 1] and [int(v) for v in m] == [1, 1, 1]      # expert 0 everywhere (tie -> lower index)
    # nothing passes the threshold: K is kept at 1 (top-1); everything passes: K = E (select-all)
    S = gi_scores(T=11, E=6)
    m1, k1 = oracle.select(S, oracle.MODE_THRESHOLD_TOPK, eps=2.0)
    mt, kt = oracle.select(S, oracle.MODE_TOPK, K=1)
    assert np.array_equal(m1, mt) and np.all(k1 == 1)
    ma, ka = oracle.select(S, oracle.MODE_THRESHOLD_TOPK, eps=0.0)
    assert np.all(ma == np.uint64(2 ** 6 - 1)) and np.all(ka == 6)


def gi_scores(T, E, seed_layer=0):
    s = gi.LayerSpec("tt", T=T, d=64, H=64, E=E, dtype="bf16", router_gain=4.0)
    x, (Wr, br) = gi.tokens(s), gi.router(s)
    return oracle.router_scores(x, Wr, br)


@pytest.mark.parametrize("normalized", [0, 1])
def test_threshold_topk_K_is_the_rounded_mean_of_the_threshold_counts(normalized):
    S = gi_scores(T=57, E=16)
    for eps in (0.02, 0.05, 0.1, 0.3):
        eps_use = eps * 16 if normalized else eps
        v = (S * np.float32(16)) if normalized else S
        counts = (v > np.float32(eps_use)).sum(axis=1)              # independent numpy thresholding
        K = int(min(16, max(1, math.floor(counts.sum() / 57 + 0.5))))
        mask, k_t = oracle.select(S, oracle.MODE_THRESHOLD_TOPK, eps=eps_use, eps_normalized=normalized)
        assert np.all(k_t == K)
        order = np.argsort(-S, axis=1, kind="stable")[:, :K]          # K highest, ties to the lower index
        want = np.zeros(57, dtype=np.uint64)
        for t in range(57):
            for e in order[t]:
                want[t] |= np.uint64(1) << np.uint64(e)
        assert np.array_equal(mask, want)
