"""Thin ctypes binding over ``libdsmoe.so``: same names as ``include/dsmoe.h``, argument marshalling
only.  Every step of the layer runs in the library's CUDA kernels; there is no fallback -- if the
shared object is missing or a call fails, an exception is raised.

Tensors are ``torch`` CUDA tensors (device memory and streams are all torch is used for); bf16
tensors are ``torch.bfloat16``, masks are ``torch.int64`` holding the uint64 bit pattern.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdsmoe.so")

F32, BF16 = 0, 1
SELECT_THRESHOLD, SELECT_TOPK, SELECT_ALL, SELECT_THRESHOLD_TOPK = 0, 1, 2, 3

EXPORTS = (
    "dsmoe_status_string", "dsmoe_workspace_size", "dsmoe_router", "dsmoe_select", "dsmoe_permute",
    "dsmoe_expert_mlp", "dsmoe_combine", "dsmoe_packed_size", "dsmoe_pack_weights",
    "dsmoe_layer_forward", "dsmoe_layer_forward_host", "dsmoe_layer_forward_host_async", "dsmoe_timing_enable", "dsmoe_timing_read",
    "dsmoe_select_static", "dsmoe_workspace_size_packed", "dsmoe_workspace_size_stages", "dsmoe_stats",
    "dsmoe_mi_loss", "dsmoe_dense_backward", "dsmoe_moa_forward",
)


class LayerDesc(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("d", ctypes.c_int32), ("H", ctypes.c_int32), ("E", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("mode", ctypes.c_int32), ("eps", ctypes.c_float),
                ("eps_normalized", ctypes.c_int32), ("K", ctypes.c_int32), ("min_k", ctypes.c_int32),
                ("out_fp32", ctypes.c_int32), ("fuse_combine", ctypes.c_int32)]


class MoaArgs(ctypes.Structure):
    _fields_ = [("n_head", ctypes.c_int32), ("n_seq", ctypes.c_int32), ("L", ctypes.c_int32), ("scale", ctypes.c_float),
                ("Kc", ctypes.c_void_p), ("Vc", ctypes.c_void_p), ("tok_seq", ctypes.c_void_p), ("pos", ctypes.c_void_p)]


class DsmoeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C-ABI library.  Raises if it has not been built (no CPU fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2404_05567_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.dsmoe_status_string.restype = ctypes.c_char_p
        L.dsmoe_status_string.argtypes = [ctypes.c_int]
        for name in EXPORTS[1:]:
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().dsmoe_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != 0:
        raise DsmoeError(code, where)


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, int):
        return ctypes.c_void_p(t)
    assert t.is_contiguous(), "dsmoe takes contiguous tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def make_desc(T, d, H, E, dtype=BF16, mode=SELECT_THRESHOLD, eps=0.0, eps_normalized=0, K=0, min_k=0,
              out_fp32=0, fuse_combine=0) -> LayerDesc:
    return LayerDesc(int(T), int(d), int(H), int(E), int(dtype), int(mode), float(eps), int(eps_normalized),
                     int(K), int(min_k), int(out_fp32), int(fuse_combine))


def width(desc: LayerDesc) -> int:
    return min(desc.K, desc.E) if desc.mode == SELECT_TOPK else desc.E


def amax(desc: LayerDesc) -> int:
    return desc.T * width(desc)


def dsmoe_workspace_size(desc: LayerDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().dsmoe_workspace_size(ctypes.byref(desc), ctypes.byref(n)), "dsmoe_workspace_size")
    return n.value


def dsmoe_workspace_size_packed(desc: LayerDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().dsmoe_workspace_size_packed(ctypes.byref(desc), ctypes.byref(n)), "dsmoe_workspace_size_packed")
    return n.value


def dsmoe_workspace_size_stages(desc: LayerDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().dsmoe_workspace_size_stages(ctypes.byref(desc), ctypes.byref(n)), "dsmoe_workspace_size_stages")
    return n.value


class SelectionStats(ctypes.Structure):
    _fields_ = [("assignments", ctypes.c_int64), ("near_threshold", ctypes.c_int64), ("zero_tokens", ctypes.c_int32),
                ("empty_experts", ctypes.c_int32), ("counts", ctypes.c_int32 * 64)]


def dsmoe_stats(desc, scores, mask, stats, stream=None):
    """``stats``: a CUDA uint8 tensor of ``ctypes.sizeof(SelectionStats)`` bytes; see ``read_stats``."""
    _check(lib().dsmoe_stats(ctypes.byref(desc), _ptr(scores), _ptr(mask), _ptr(stats), _stream(stream)), "dsmoe_stats")


def read_stats(stats) -> dict:
    """Copies the device struct back (synchronises) and returns it as a dict."""
    raw = bytes(stats.cpu().numpy().tobytes())
    st = SelectionStats.from_buffer_copy(raw)
    return dict(assignments=int(st.assignments), near_threshold=int(st.near_threshold), zero_tokens=int(st.zero_tokens),
                empty_experts=int(st.empty_experts), counts=[int(c) for c in st.counts])


def dsmoe_packed_size(desc: LayerDesc) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().dsmoe_packed_size(ctypes.byref(desc), ctypes.byref(n)), "dsmoe_packed_size")
    return n.value


def dsmoe_router(desc, x, Wr, br, scores, stream=None):
    _check(lib().dsmoe_router(ctypes.byref(desc), _ptr(x), _ptr(Wr), _ptr(br), _ptr(scores), _stream(stream)),
           "dsmoe_router")


def dsmoe_select(desc, scores, mask, k_t, counts, offsets, workspace, stream=None):
    _check(lib().dsmoe_select(ctypes.byref(desc), _ptr(scores), _ptr(mask), _ptr(k_t), _ptr(counts), _ptr(offsets),
                              _ptr(workspace), ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                              _stream(stream)), "dsmoe_select")


def dsmoe_permute(desc, x, scores, mask, offsets, row_token, row_gate, token_rows, xp, workspace, stream=None):
    _check(lib().dsmoe_permute(ctypes.byref(desc), _ptr(x), _ptr(scores), _ptr(mask), _ptr(offsets), _ptr(row_token),
                               _ptr(row_gate), _ptr(token_rows), _ptr(xp), _ptr(workspace),
                               ctypes.c_size_t(workspace.numel() if workspace is not None else 0), _stream(stream)),
           "dsmoe_permute")


def dsmoe_expert_mlp(desc, xp, W1, W2, packed, offsets, yp, workspace, dev_status=None, stream=None):
    _check(lib().dsmoe_expert_mlp(ctypes.byref(desc), _ptr(xp), _ptr(W1), _ptr(W2), _ptr(packed), _ptr(offsets),
                                  _ptr(yp), _ptr(workspace),
                                  ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                                  _ptr(dev_status), _stream(stream)), "dsmoe_expert_mlp")


def dsmoe_combine(desc, yp, row_gate, token_rows, k_t, out, stream=None):
    _check(lib().dsmoe_combine(ctypes.byref(desc), _ptr(yp), _ptr(row_gate), _ptr(token_rows), _ptr(k_t), _ptr(out),
                               _stream(stream)), "dsmoe_combine")


def dsmoe_pack_weights(desc, W1, W2, packed, stream=None):
    _check(lib().dsmoe_pack_weights(ctypes.byref(desc), _ptr(W1), _ptr(W2), _ptr(packed), _stream(stream)),
           "dsmoe_pack_weights")


def dsmoe_layer_forward(desc, x, Wr, br, W1, W2, packed, out, mask_out, counts_out, workspace, dev_status=None,
                        stream=None):
    _check(lib().dsmoe_layer_forward(ctypes.byref(desc), _ptr(x), _ptr(Wr), _ptr(br), _ptr(W1), _ptr(W2),
                                     _ptr(packed), _ptr(out), _ptr(mask_out), _ptr(counts_out), _ptr(workspace),
                                     ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                                     _ptr(dev_status), _stream(stream)), "dsmoe_layer_forward")


def dsmoe_layer_forward_host(desc, x_host, x_dev, Wr, br, W1, W2, packed, out_dev, out_host, workspace,
                             dev_status=None, stream=None):
    """``x_host`` / ``out_host`` are CPU tensors (pinned for full copy speed); the call returns after
    the result has landed in ``out_host``."""
    _check(lib().dsmoe_layer_forward_host(ctypes.byref(desc), _ptr(x_host), _ptr(x_dev), _ptr(Wr), _ptr(br),
                                          _ptr(W1), _ptr(W2), _ptr(packed), _ptr(out_dev), _ptr(out_host),
                                          _ptr(workspace),
                                          ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                                          _ptr(dev_status), _stream(stream)), "dsmoe_layer_forward_host")


def dsmoe_layer_forward_host_async(desc, x_host, x_dev, Wr, br, W1, W2, packed, out_dev, out_host, workspace,
                                   dev_status=None, stream=None):
    """As ``dsmoe_layer_forward_host`` without the final wait: ``out_host`` may be read once the stream has
    been waited for."""
    _check(lib().dsmoe_layer_forward_host_async(ctypes.byref(desc), _ptr(x_host), _ptr(x_dev), _ptr(Wr), _ptr(br),
                                                _ptr(W1), _ptr(W2), _ptr(packed), _ptr(out_dev), _ptr(out_host),
                                                _ptr(workspace),
                                                ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                                                _ptr(dev_status), _stream(stream)), "dsmoe_layer_forward_host_async")


def dsmoe_mi_loss(desc, scores, loss3, grad, workspace, stream=None):
    _check(lib().dsmoe_mi_loss(ctypes.byref(desc), _ptr(scores), _ptr(loss3), _ptr(grad), _ptr(workspace),
                               ctypes.c_size_t(workspace.numel() if workspace is not None else 0), _stream(stream)),
           "dsmoe_mi_loss")


def dsmoe_dense_backward(desc, x, W1, W2, packed, scores, mask, dO, dS, dA, workspace, dev_status=None, stream=None):
    _check(lib().dsmoe_dense_backward(ctypes.byref(desc), _ptr(x), _ptr(W1), _ptr(W2), _ptr(packed), _ptr(scores),
                                      _ptr(mask), _ptr(dO), _ptr(dS), _ptr(dA), _ptr(workspace),
                                      ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                                      _ptr(dev_status), _stream(stream)), "dsmoe_dense_backward")


def dsmoe_moa_forward(desc, n_head, scale, Kc, Vc, tok_seq, pos, x, Wr, br, packed, out, mask_out, counts_out, workspace,
                      dev_status=None, stream=None):
    """Mixture-of-attention-heads layer (Eq. 7-8).  Kc, Vc: [n_seq, n_head, L, d_head] bf16 tensors."""
    n_seq, nh, L, _ = Kc.shape
    assert nh == n_head and Vc.shape == Kc.shape
    args = MoaArgs(int(n_head), int(n_seq), int(L), float(scale), _ptr(Kc), _ptr(Vc), _ptr(tok_seq), _ptr(pos))
    _check(lib().dsmoe_moa_forward(ctypes.byref(desc), ctypes.byref(args), _ptr(x), _ptr(Wr), _ptr(br), _ptr(packed),
                                   _ptr(out), _ptr(mask_out), _ptr(counts_out), _ptr(workspace),
                                   ctypes.c_size_t(workspace.numel() if workspace is not None else 0),
                                   _ptr(dev_status), _stream(stream)), "dsmoe_moa_forward")


def dsmoe_timing_enable(n_pairs: int):
    _check(lib().dsmoe_timing_enable(ctypes.c_int(int(n_pairs))), "dsmoe_timing_enable")


def dsmoe_timing_read(n_max: int):
    """Durations (ms) of the timed launches since the ring was enabled or last read, in launch order."""
    buf = (ctypes.c_float * max(n_max, 1))()
    n = ctypes.c_int(0)
    _check(lib().dsmoe_timing_read(buf, ctypes.c_int(n_max), ctypes.byref(n)), "dsmoe_timing_read")
    return [float(buf[i]) for i in range(n.value)]


def dsmoe_select_static(desc, scores, mask, k_t, counts, offsets, stream=None):
    """dsmoe_select for callers that cannot allocate: no workspace argument, the scratch is a fixed
    array inside the library (limit ceil(T/32)*E <= 131072, else status 3)."""
    _check(lib().dsmoe_select_static(ctypes.byref(desc), _ptr(scores), _ptr(mask), _ptr(k_t), _ptr(counts),
                                     _ptr(offsets), _stream(stream)), "dsmoe_select_static")
