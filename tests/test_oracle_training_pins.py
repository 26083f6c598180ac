"""Pins for the oracle's training-side functions: the mutual-information loss of the router (Eq. 4-6) and the
gradients of dense training (Eq. 2, Eq. 3).  Closed forms, a library routine, finite differences of the forward
oracle, and a separately written numpy restatement."""
import math

import numpy as np
import pytest
from scipy.special import erf
from scipy.stats import entropy

import dsmoe_inputs as gi
import oracle


def _rand(name, shape, scale=1.0, dtype="f32", seed=13):
    return gi.normal(seed, name, shape, scale, dtype)


def _softmax_rows(name, T, E, gain=1.5):
    raw = _rand(name, (T, E), gain).astype(np.float64)
    p = np.exp(raw - raw.max(1, keepdims=True))
    return (p / p.sum(1, keepdims=True)).astype(np.float32)


# ---------------------------------------------------------------- mutual-information loss (Eq. 4-6)

@pytest.mark.parametrize("N", [2, 8, 32, 64])
def test_mi_loss_closed_forms(N):
    T = 3 * N
    uniform = np.full((T, N), 1.0 / N, dtype=np.float32)
    L, He, Hc = oracle.mi_loss(uniform)
    # every token spreads evenly: both entropies are ln N and the loss (minus the mutual information) is 0
    assert He == pytest.approx(math.log(N), rel=1e-6) and Hc == pytest.approx(math.log(N), rel=1e-6)
    assert L == pytest.approx(0.0, abs=1e-6)
    balanced = np.zeros((T, N), dtype=np.float32)
    balanced[np.arange(T), np.arange(T) % N] = 1.0
    L, He, Hc = oracle.mi_loss(balanced)
    # one-hot routers that share the load evenly: H(e|X) = 0, H(e) = ln N, the minimum of the loss
    assert Hc == 0.0 and He == pytest.approx(math.log(N), rel=1e-12) and L == pytest.approx(-math.log(N), rel=1e-12)
    collapsed = np.zeros((T, N), dtype=np.float32)
    collapsed[:, N // 2] = 1.0
    assert oracle.mi_loss(collapsed) == (0.0, 0.0, 0.0)       # every token on one expert: no information either way


def test_mi_loss_matches_library_entropies_and_is_minus_a_mutual_information():
    T, N = 211, 32
    S = _softmax_rows("mi", T, N)
    L, He, Hc = oracle.mi_loss(S)
    Sd = S.astype(np.float64)
    assert He == pytest.approx(float(entropy(Sd.mean(axis=0))), rel=1e-9)          # scipy renormalises: sums are 1 +- 1e-7
    assert Hc == pytest.approx(float(np.mean([entropy(row) for row in Sd])), rel=1e-6)
    assert L == pytest.approx(Hc - He, rel=1e-12)
    assert L <= 1e-9                                                                # I(e;X) >= 0
    # the marginal is a mean over tokens: permuting the tokens changes nothing, duplicating the batch neither
    perm = gi.permutation(3, "mi.perm", T)
    assert oracle.mi_loss(S[perm]) == pytest.approx((L, He, Hc), rel=1e-12)
    assert oracle.mi_loss(np.concatenate([S, S])) == pytest.approx((L, He, Hc), rel=1e-12)


def test_mi_loss_gradient_against_central_differences():
    T, N = 9, 5
    S = _softmax_rows("mig", T, N, 1.0)
    _, _, _, grad = oracle.mi_loss(S, want_grad=True)
    h = 2.0 ** -10                      # exactly representable in fp32 next to scores of order 0.1
    for t, e in [(0, 0), (3, 4), (8, 2), (5, 1)]:
        Sp, Sm = S.copy(), S.copy()
        Sp[t, e] += np.float32(h)
        Sm[t, e] -= np.float32(h)
        step = float(Sp[t, e]) - float(Sm[t, e])
        fd = (oracle.mi_loss(Sp)[0] - oracle.mi_loss(Sm)[0]) / step
        assert grad[t, e] == pytest.approx(fd, rel=2e-4, abs=1e-7)


# ---------------------------------------------------------------- gradients of dense training (Eq. 2, Eq. 3)

def _tiny(dtype="f32"):
    T, d, H, E = 6, 12, 10, 5
    x = _rand("bx", (T, d), 1.0, dtype)
    W1 = _rand("bW1", (E, d, H), 0.3, dtype)
    W2 = _rand("bW2", (E, H, d), 0.3, dtype)
    dO = _rand("bdO", (T, d), 1.0, dtype)
    S = _softmax_rows("bS", T, E, 1.0)
    return x, W1, W2, dO, S


def test_grad_S_is_the_derivative_of_the_dense_forward():
    """L = <O, dO> with O = sum_j S_j e_j(X) (every expert, Eq. 3's forward) is linear in S: central differences of
    the forward oracle are exact up to rounding."""
    x, W1, W2, dO, S = _tiny()
    T, E = S.shape
    every = np.full(T, (1 << E) - 1, dtype=np.uint64)
    dS, _ = oracle.dense_backward(x, W1, W2, S, dO)
    h = np.float32(2.0 ** -6)
    for t, j in [(0, 0), (2, 3), (5, 4), (4, 1)]:
        Sp, Sm = S.copy(), S.copy()
        Sp[t, j] += h
        Sm[t, j] -= h
        Lp = float((oracle.layer(x, W1, W2, Sp, every) * dO.astype(np.float64)).sum())
        Lm = float((oracle.layer(x, W1, W2, Sm, every) * dO.astype(np.float64)).sum())
        fd = (Lp - Lm) / (float(Sp[t, j]) - float(Sm[t, j]))
        assert dS[t, j] == pytest.approx(fd, rel=1e-9, abs=1e-12)


def test_sparse_training_gradient_is_the_dense_one_masked():
    """Eq. 2 = Eq. 3 (x) M, and it is the derivative of the sparse forward (Eq. 1 with the same mask)."""
    x, W1, W2, dO, S = _tiny()
    mask, _ = oracle.select(S, oracle.MODE_TOPK, K=2)
    dS_dense, dA_dense = oracle.dense_backward(x, W1, W2, S, dO)
    dS_sparse, dA_sparse = oracle.dense_backward(x, W1, W2, S, dO, mask=mask)
    M = np.array([[(int(m) >> e) & 1 for e in range(S.shape[1])] for m in mask], dtype=np.float64)
    assert np.array_equal(dS_sparse, dS_dense * M)
    assert np.array_equal(dA_sparse, dA_dense * M[:, :, None])
    h = np.float32(2.0 ** -6)
    for t in range(S.shape[0]):
        for j in range(S.shape[1]):
            Sp, Sm = S.copy(), S.copy()
            Sp[t, j] += h
            Sm[t, j] -= h
            Lp = float((oracle.layer(x, W1, W2, Sp, mask) * dO.astype(np.float64)).sum())
            Lm = float((oracle.layer(x, W1, W2, Sm, mask) * dO.astype(np.float64)).sum())
            fd = (Lp - Lm) / (float(Sp[t, j]) - float(Sm[t, j]))
            assert dS_sparse[t, j] == pytest.approx(fd, rel=1e-9, abs=1e-12)


def _np_gelu(v):
    return 0.5 * v * (1.0 + erf(v / math.sqrt(2.0)))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gradients_against_a_numpy_restatement(dtype):
    x, W1, W2, dO, S = _tiny(dtype)
    dS, dA = oracle.dense_backward(x, W1, W2, S, dO)
    xf, W1f, W2f, dOf = (gi.as_f32(a).astype(np.float64) for a in (x, W1, W2, dO))
    a = _np_gelu(np.einsum("td,edh->teh", xf, W1f))                  # hidden activations of every expert
    y = np.einsum("teh,ehd->ted", a, W2f)                            # e_j(X)
    np.testing.assert_allclose(dS, np.einsum("ted,td->te", y, dOf), rtol=1e-10, atol=1e-12)
    want_dA = S.astype(np.float64)[:, :, None] * np.einsum("td,ehd->teh", dOf, W2f)   # (S_j dO) W2_j^T
    np.testing.assert_allclose(dA, want_dA, rtol=1e-10, atol=1e-12)
    # the two halves of Eq. 3 meet: <a_j, dA_j> = S_j <e_j(X), dO> = S_j dS_j
    np.testing.assert_allclose(np.einsum("teh,teh->te", a, dA), S.astype(np.float64) * dS, rtol=1e-9, atol=1e-12)


def test_grad_at_the_hidden_activation_against_central_differences():
    """dA is the derivative of L = <O, dO> with respect to the hidden activation a_j of one expert: a numpy layer with
    a_j nudged along a direction u gives the same number."""
    x, W1, W2, dO, S = _tiny()
    _, dA = oracle.dense_backward(x, W1, W2, S, dO)
    xf, W1f, W2f, dOf, Sf = (a.astype(np.float64) for a in (x, W1, W2, dO, S))
    u = _rand("u", (W1.shape[2],)).astype(np.float64)

    def loss(theta, t, j):
        a = _np_gelu(np.einsum("td,edh->teh", xf, W1f))
        a[t, j] += theta * u
        O = np.einsum("te,teh,ehd->td", Sf, a, W2f)
        return float((O * dOf).sum())

    for t, j in [(0, 0), (3, 2), (5, 4)]:
        fd = (loss(1e-3, t, j) - loss(-1e-3, t, j)) / 2e-3
        assert float(dA[t, j] @ u) == pytest.approx(fd, rel=1e-8)


def test_token_subset_and_token_independence():
    x, W1, W2, dO, S = _tiny()
    dS, dA = oracle.dense_backward(x, W1, W2, S, dO)
    ids = np.array([4, 1], dtype=np.int64)
    dS2, dA2 = oracle.dense_backward(x, W1, W2, S, dO, token_ids=ids)
    assert np.array_equal(dS2, dS[ids]) and np.array_equal(dA2, dA[ids])
