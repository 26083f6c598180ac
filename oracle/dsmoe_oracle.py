"""ctypes wrapper around ``dsmoe_oracle.c`` (plain C, fp64) -- TEST INFRASTRUCTURE ONLY.

Every function here is the paper's definition evaluated token by token in double
precision; see the header of ``dsmoe_oracle.c`` for the passages followed and the
readings taken where the paper is silent.  bf16 tensors are passed as uint16 bit
patterns, fp32 tensors as float32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dsmoe_oracle.c")
_LIB = os.path.join(_HERE, "libdsmoe_oracle.so")
_lib = None

MODE_THRESHOLD, MODE_TOPK, MODE_ALL, MODE_THRESHOLD_TOPK = 0, 1, 2, 3

__all__ = [
    "build", "router_scores", "select", "group", "layer", "expert_rows", "combine", "mi_loss", "dense_backward", "moa_layer",
    "num_threads", "MODE_THRESHOLD", "MODE_TOPK", "MODE_ALL", "MODE_THRESHOLD_TOPK",
]


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return 0
    if a.dtype == np.uint16:
        return 1
    raise TypeError(f"expected float32 or uint16 (bf16 bits), got {a.dtype}")


def _c(a, dtype=None):
    return np.ascontiguousarray(a) if dtype is None else np.ascontiguousarray(a, dtype=dtype)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def router_scores(x, Wr, br=None) -> np.ndarray:
    """S = softmax(x.Wr + b) per token (Eq. 1); double arithmetic, one rounding to fp32."""
    x, Wr = _c(x), _c(Wr, np.float32)
    br = None if br is None else _c(br, np.float32)
    T, d = x.shape
    E = Wr.shape[1]
    assert Wr.shape[0] == d and E <= 64
    S = np.empty((T, E), dtype=np.float32)
    _load().oracle_router_scores(_p(x), _dtype_code(x), _p(Wr), _p(br),
                                 ctypes.c_int64(T), ctypes.c_int64(d), ctypes.c_int64(E), _p(S))
    return S


def select(scores, mode, eps=0.0, eps_normalized=0, K=0, min_k=0):
    """(mask uint64[T], k_t int32[T]) from fp32 scores ("Sparse Inference" paragraph)."""
    S = _c(scores, np.float32)
    T, E = S.shape
    mask = np.zeros(T, dtype=np.uint64)
    k_t = np.zeros(T, dtype=np.int32)
    _load().oracle_select(_p(S), ctypes.c_int64(T), ctypes.c_int64(E), ctypes.c_int(mode),
                          ctypes.c_float(eps), ctypes.c_int(eps_normalized), ctypes.c_int(K),
                          ctypes.c_int(min_k), _p(mask), _p(k_t))
    return mask, k_t


def group(mask, scores, width=None):
    """Grouping of (token, expert) assignments by expert, canonical order.

    Returns dict(counts[E], offsets[E+1], row_token[A], row_gate[A], row_expert[A],
    token_rows[T,width]); rows ascend by token inside an expert, token_rows lists a
    token's rows in ascending expert order and is -1 past k_t.
    """
    S = _c(scores, np.float32)
    mask = _c(mask, np.uint64)
    T, E = S.shape
    width = E if width is None else int(width)
    amax = T * E
    counts = np.zeros(E, np.int32)
    offsets = np.zeros(E + 1, np.int32)
    row_token = np.full(amax, -1, np.int32)
    row_gate = np.zeros(amax, np.float32)
    row_expert = np.full(amax, -1, np.int32)
    token_rows = np.full((T, width), -1, np.int32)
    _load().oracle_group(_p(mask), _p(S), ctypes.c_int64(T), ctypes.c_int64(E),
                         ctypes.c_int64(width), _p(counts), _p(offsets), _p(row_token),
                         _p(row_gate), _p(row_expert), _p(token_rows))
    A = int(offsets[E])
    return dict(counts=counts, offsets=offsets, row_token=row_token[:A], row_gate=row_gate[:A],
                row_expert=row_expert[:A], token_rows=token_rows, A=A)


def layer(x, W1, W2, scores, mask, token_ids=None) -> np.ndarray:
    """O[t] = sum_{e selected} S[t,e] * GeLU(x[t].W1[e]).W2[e]  (Eq. 1), float64.

    ``token_ids`` restricts the evaluation to those tokens (rows of the result follow it).
    """
    x, W1, W2 = _c(x), _c(W1), _c(W2)
    S = _c(scores, np.float32)
    mask = _c(mask, np.uint64)
    T, d = x.shape
    E, d1, H = W1.shape
    assert d1 == d and W2.shape == (E, H, d) and S.shape == (T, E)
    dt = _dtype_code(x)
    assert _dtype_code(W1) == dt and _dtype_code(W2) == dt
    ids = None if token_ids is None else _c(token_ids, np.int64)
    n = T if ids is None else ids.shape[0]
    out = np.empty((n, d), dtype=np.float64)
    _load().oracle_layer(_p(x), _p(W1), _p(W2), dt, _p(S), _p(mask), _p(ids), ctypes.c_int64(n),
                         ctypes.c_int64(d), ctypes.c_int64(H), ctypes.c_int64(E), _p(out))
    return out


def moa_layer(x, Wq, Wo, Kc, Vc, scores, mask, pos, n_head, scale, tok_seq=None, token_ids=None) -> np.ndarray:
    """Mixture-of-attention-heads layer (Eq. 7-8), float64:
    O[t] = sum_{i selected} S[t,i] sum_j softmax(scale Q_ij K_j^T) V_j Wo_ij over keys 0..pos[t] of the token's sequence.

    Wq [E, d, n_head*dh], Wo [E, n_head*dh, d], Kc and Vc [n_seq, n_head, L, dh]."""
    x, Wq, Wo, Kc, Vc = _c(x), _c(Wq), _c(Wo), _c(Kc), _c(Vc)
    S = _c(scores, np.float32)
    mask = _c(mask, np.uint64)
    pos = _c(pos, np.int32)
    T, d = x.shape
    E, d1, H = Wq.shape
    n_seq, nh, L, dh = Kc.shape
    assert d1 == d and Wo.shape == (E, H, d) and S.shape == (T, E) and nh == n_head and H == n_head * dh
    assert Vc.shape == Kc.shape and pos.shape == (T,) and pos.min(initial=0) >= 0 and pos.max(initial=0) < L
    dt = _dtype_code(x)
    assert all(_dtype_code(a) == dt for a in (Wq, Wo, Kc, Vc))
    seq = None if tok_seq is None else _c(tok_seq, np.int32)
    assert seq is None or (seq.shape == (T,) and seq.min(initial=0) >= 0 and seq.max(initial=0) < n_seq)
    ids = None if token_ids is None else _c(token_ids, np.int64)
    n = T if ids is None else ids.shape[0]
    out = np.empty((n, d), dtype=np.float64)
    _load().oracle_moa_layer(_p(x), _p(Wq), _p(Wo), _p(Kc), _p(Vc), dt, _p(S), _p(mask), _p(seq), _p(pos), _p(ids),
                             ctypes.c_int64(n), ctypes.c_int64(d), ctypes.c_int64(n_head), ctypes.c_int64(dh),
                             ctypes.c_int64(E), ctypes.c_int64(L), ctypes.c_double(scale), _p(out))
    return out


def expert_rows(xp, W1, W2, row_expert, rows=None) -> np.ndarray:
    """yp[r] = e_{row_expert[r]}(xp[r]) for grouped rows, float64 [len(rows), d]."""
    xp, W1, W2 = _c(xp), _c(W1), _c(W2)
    row_expert = _c(row_expert, np.int32)
    E, d, H = W1.shape
    dt = _dtype_code(xp)
    ids = None if rows is None else _c(rows, np.int64)
    n = xp.shape[0] if ids is None else ids.shape[0]
    yp = np.empty((n, d), dtype=np.float64)
    _load().oracle_expert_rows(_p(xp), _p(W1), _p(W2), dt, _p(row_expert), _p(ids),
                               ctypes.c_int64(n), ctypes.c_int64(d), ctypes.c_int64(H), _p(yp))
    return yp


def mi_loss(scores, want_grad: bool = False):
    """Mutual-information loss of the router (Eq. 4-6): returns (L_MI, H(e), mean H(e|X)) and, with
    ``want_grad``, also dL_MI/dS as float64 [T,E]."""
    S = _c(scores, np.float32)
    T, E = S.shape
    out3 = np.zeros(3, dtype=np.float64)
    grad = np.empty((T, E), dtype=np.float64) if want_grad else None
    _load().oracle_mi_loss(_p(S), ctypes.c_int64(T), ctypes.c_int64(E), _p(out3), _p(grad))
    res = (float(out3[0]), float(out3[1]), float(out3[2]))
    return res + (grad,) if want_grad else res


def dense_backward(x, W1, W2, scores, dO, mask=None, token_ids=None, want_dA: bool = True):
    """Gradients of dense training (Eq. 3; Eq. 2 with ``mask``): dS[n,E] = <e_j(x), dO> and dA[n,E,H] =
    (S_j dO).W2[j]^T, the gradient at the experts' hidden activations.  float64."""
    x, W1, W2, dO = _c(x), _c(W1), _c(W2), _c(dO)
    S = _c(scores, np.float32)
    T, d = x.shape
    E, d1, H = W1.shape
    assert d1 == d and W2.shape == (E, H, d) and S.shape == (T, E) and dO.shape == (T, d)
    dt = _dtype_code(x)
    assert _dtype_code(W1) == dt and _dtype_code(W2) == dt and _dtype_code(dO) == dt
    mask = None if mask is None else _c(mask, np.uint64)
    ids = None if token_ids is None else _c(token_ids, np.int64)
    n = T if ids is None else ids.shape[0]
    dS = np.empty((n, E), dtype=np.float64)
    dA = np.empty((n, E, H), dtype=np.float64) if want_dA else None
    _load().oracle_dense_backward(_p(x), _p(W1), _p(W2), dt, _p(S), _p(mask), _p(dO), _p(ids), ctypes.c_int64(n),
                                  ctypes.c_int64(d), ctypes.c_int64(H), ctypes.c_int64(E), _p(dS), _p(dA))
    return dS, dA


def combine(yp, row_gate, token_rows) -> np.ndarray:
    """out[t] = sum_i row_gate[r_i] * yp[r_i] over token t's rows, float64 [T, d]."""
    yp = _c(yp, np.float32)
    row_gate = _c(row_gate, np.float32)
    token_rows = _c(token_rows, np.int32)
    T, width = token_rows.shape
    d = yp.shape[1]
    out = np.empty((T, d), dtype=np.float64)
    _load().oracle_combine(_p(yp), _p(row_gate), _p(token_rows), ctypes.c_int64(T),
                           ctypes.c_int64(width), ctypes.c_int64(d), _p(out))
    return out
