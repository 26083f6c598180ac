"""Pins for the oracle's mixture-of-attention-heads layer (Eq. 7-8): special cases with closed forms, an einsum
restatement through a library softmax, a pure-Python brute force, and the invariances the definition implies."""
import numpy as np
import pytest
from scipy.special import softmax

import dsmoe_inputs as gi
import oracle


def _rand(name, shape, scale=1.0, seed=29):
    return gi.normal(seed, name, shape, scale, "f32")


def _case(T=6, d=12, E=3, nh=2, dh=4, L=7, n_seq=2, seed=29):
    x = _rand("moa.x", (T, d), 1.0, seed)
    Wq = _rand("moa.Wq", (E, d, nh * dh), 0.4, seed)
    Wo = _rand("moa.Wo", (E, nh * dh, d), 0.4, seed)
    Kc = _rand("moa.K", (n_seq, nh, L, dh), 1.0, seed)
    Vc = _rand("moa.V", (n_seq, nh, L, dh), 1.0, seed)
    raw = _rand("moa.S", (T, E), 1.0, seed).astype(np.float64)
    S = softmax(raw, axis=1).astype(np.float32)
    pos = (np.arange(T) * 3 % L).astype(np.int32)
    seq = (np.arange(T) % n_seq).astype(np.int32)
    return x, Wq, Wo, Kc, Vc, S, pos, seq


def _einsum_reference(x, Wq, Wo, Kc, Vc, S, mask, pos, seq, nh, scale):
    """The same layer written token by token with einsum and scipy's softmax."""
    T, d = x.shape
    E = Wq.shape[0]
    dh = Kc.shape[-1]
    out = np.zeros((T, d))
    for t in range(T):
        K = Kc[seq[t], :, :pos[t] + 1].astype(np.float64)          # [nh, l, dh]
        V = Vc[seq[t], :, :pos[t] + 1].astype(np.float64)
        for i in range(E):
            if not (int(mask[t]) >> i) & 1:
                continue
            Q = (x[t].astype(np.float64) @ Wq[i].astype(np.float64)).reshape(nh, dh)
            P = softmax(scale * np.einsum("jc,jlc->jl", Q, K), axis=1)
            A = np.einsum("jl,jlc->jc", P, V).reshape(nh * dh)
            out[t] += float(S[t, i]) * (A @ Wo[i].astype(np.float64))
    return out


def test_moa_against_einsum_and_library_softmax():
    x, Wq, Wo, Kc, Vc, S, pos, seq = _case()
    mask = np.array([0b111, 0b001, 0b110, 0b010, 0b101, 0b000], dtype=np.uint64)
    got = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, pos, 2, 0.5, tok_seq=seq)
    ref = _einsum_reference(x, Wq, Wo, Kc, Vc, S, mask, pos, seq, 2, 0.5)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-13)
    assert np.all(got[5] == 0.0)                          # no expert selected: the empty sum of Eq. 8


def test_moa_brute_force_loops():
    T, d, E, nh, dh, L = 3, 4, 2, 2, 2, 3
    x, Wq, Wo, Kc, Vc, S, pos, seq = _case(T, d, E, nh, dh, L, 1, seed=31)
    mask = np.array([0b11, 0b10, 0b01], dtype=np.uint64)
    got = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, pos, nh, 1.0)
    for t in range(T):
        o = [0.0] * d
        for i in range(E):
            if not (int(mask[t]) >> i) & 1:
                continue
            for j in range(nh):
                q = [sum(float(x[t, k]) * float(Wq[i, k, j * dh + c]) for k in range(d)) for c in range(dh)]
                logit = [sum(q[c] * float(Kc[0, j, l, c]) for c in range(dh)) for l in range(pos[t] + 1)]
                m = max(logit)
                w = [np.exp(v - m) for v in logit]
                den = sum(w)
                a = [sum(w[l] / den * float(Vc[0, j, l, c]) for l in range(pos[t] + 1)) for c in range(dh)]
                for c2 in range(d):
                    o[c2] += float(S[t, i]) * sum(a[c] * float(Wo[i, j * dh + c, c2]) for c in range(dh))
        assert np.allclose(got[t], o, rtol=1e-12, atol=1e-14)


def test_moa_zero_queries_average_the_values():
    """Wq = 0: every softmax is uniform over the visible keys, so a_ij is the mean of V_j[0..pos]."""
    x, Wq, Wo, Kc, Vc, S, pos, seq = _case()
    mask = np.full(x.shape[0], 0b111, dtype=np.uint64)
    got = oracle.moa_layer(x, 0 * Wq, Wo, Kc, Vc, S, mask, pos, 2, 0.7, tok_seq=seq)
    for t in range(x.shape[0]):
        mean_v = Vc[seq[t], :, :pos[t] + 1].astype(np.float64).mean(axis=1).reshape(-1)      # [nh*dh]
        ref = sum(float(S[t, i]) * (mean_v @ Wo[i].astype(np.float64)) for i in range(3))
        assert np.allclose(got[t], ref, rtol=1e-12, atol=1e-13)


def test_moa_single_visible_key_passes_its_value_through():
    x, Wq, Wo, Kc, Vc, S, pos, seq = _case()
    pos0 = np.zeros_like(pos)
    mask = np.full(x.shape[0], 0b011, dtype=np.uint64)
    got = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, pos0, 2, 3.0, tok_seq=seq)
    for t in range(x.shape[0]):
        v0 = Vc[seq[t], :, 0].astype(np.float64).reshape(-1)
        ref = sum(float(S[t, i]) * (v0 @ Wo[i].astype(np.float64)) for i in range(2))
        assert np.allclose(got[t], ref, rtol=1e-12, atol=1e-13)


def test_moa_uniform_router_is_grouped_query_attention():
    """Every expert selected with score 1/N: (1/N) x plain grouped-query attention with N * n_head query heads on n_head
    key/value heads and one concatenated output projection."""
    x, Wq, Wo, Kc, Vc, _, pos, seq = _case(T=5, d=8, E=4, nh=2, dh=4, L=6, n_seq=1)
    T, d = x.shape
    E, nh, dh = 4, 2, 4
    S = np.full((T, E), 1.0 / E, dtype=np.float32)
    mask = np.full(T, (1 << E) - 1, dtype=np.uint64)
    got = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, pos, nh, 0.5)
    Wq_cat = np.concatenate([Wq[i] for i in range(E)], axis=1).astype(np.float64)           # [d, E*nh*dh]
    Wo_cat = np.concatenate([Wo[i] for i in range(E)], axis=0).astype(np.float64)           # [E*nh*dh, d]
    for t in range(T):
        Q = (x[t].astype(np.float64) @ Wq_cat).reshape(E * nh, dh)
        heads = []
        for h in range(E * nh):
            j = h % nh                                                                     # its key/value head
            K, V = Kc[0, j, :pos[t] + 1].astype(np.float64), Vc[0, j, :pos[t] + 1].astype(np.float64)
            heads.append(softmax(0.5 * (K @ Q[h])) @ V)
        ref = np.concatenate(heads) @ Wo_cat / E
        assert np.allclose(got[t], ref, rtol=1e-12, atol=1e-13)


def test_moa_invariances():
    x, Wq, Wo, Kc, Vc, S, pos, seq = _case()
    T = x.shape[0]
    mask = np.array([0b111, 0b011, 0b110, 0b100, 0b101, 0b010], dtype=np.uint64)
    base = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, pos, 2, 0.5, tok_seq=seq)
    # keys and values past a token's position do not exist for it
    K2, V2 = Kc.copy(), Vc.copy()
    for s in range(Kc.shape[0]):
        worst = max(int(p) for p, q in zip(pos, seq) if q == s)
        K2[s, :, worst + 1:] = 77.0
        V2[s, :, worst + 1:] = -55.0
    assert np.array_equal(oracle.moa_layer(x, Wq, Wo, K2, V2, S, mask, pos, 2, 0.5, tok_seq=seq), base)
    # attention does not care about the order of the visible keys: permute keys and values of a full cache together
    full = np.full(T, Kc.shape[2] - 1, dtype=np.int32)
    perm = np.array([3, 0, 6, 2, 5, 1, 4])
    a = oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, full, 2, 0.5, tok_seq=seq)
    b = oracle.moa_layer(x, Wq, Wo, Kc[:, :, perm], Vc[:, :, perm], S, mask, full, 2, 0.5, tok_seq=seq)
    assert np.allclose(a, b, rtol=1e-12, atol=1e-13)
    # a constant added to every key of a head shifts all its logits alike: nothing changes
    c = oracle.moa_layer(x, Wq, Wo, Kc + 0.0, Vc, S, mask, pos, 2, 0.0, tok_seq=seq)            # scale 0: uniform weights
    d0 = oracle.moa_layer(x, 0 * Wq, Wo, Kc, Vc, S, mask, pos, 2, 0.5, tok_seq=seq)
    assert np.allclose(c, d0, rtol=1e-12, atol=1e-13)
    # linear in the values, in the output projection and in the scores
    assert np.allclose(oracle.moa_layer(x, Wq, Wo, Kc, 2 * Vc, S, mask, pos, 2, 0.5, tok_seq=seq), 2 * base, rtol=1e-12)
    assert np.allclose(oracle.moa_layer(x, Wq, -4 * Wo, Kc, Vc, S, mask, pos, 2, 0.5, tok_seq=seq), -4 * base, rtol=1e-12, atol=1e-14)
    assert np.allclose(oracle.moa_layer(x, Wq, Wo, Kc, Vc, (0.5 * S).astype(np.float32), mask, pos, 2, 0.5, tok_seq=seq),
                       0.5 * base, rtol=1e-12)
    # tokens are independent, and token_ids picks rows
    ids = np.array([4, 1, 1, 0], dtype=np.int64)
    assert np.array_equal(oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask, pos, 2, 0.5, tok_seq=seq, token_ids=ids), base[ids])
    # one expert at a time adds up to all of them
    parts = sum(oracle.moa_layer(x, Wq, Wo, Kc, Vc, S, mask & np.uint64(1 << i), pos, 2, 0.5, tok_seq=seq) for i in range(3))
    assert np.allclose(parts, base, rtol=1e-12, atol=1e-13)


def test_moa_bf16_inputs_are_read_as_their_values():
    x, Wq, Wo, Kc, Vc, S, pos, seq = _case()
    mask = np.full(x.shape[0], 0b101, dtype=np.uint64)
    as16 = [gi.f32_to_bf16(a) for a in (x, Wq, Wo, Kc, Vc)]
    as32 = [gi.bf16_to_f32(a) for a in as16]
    a = oracle.moa_layer(*as16, S, mask, pos, 2, 0.5, tok_seq=seq)
    b = oracle.moa_layer(*as32, S, mask, pos, 2, 0.5, tok_seq=seq)
    assert np.array_equal(a, b)
