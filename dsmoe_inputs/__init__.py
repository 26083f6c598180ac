"""Seeded synthetic inputs for the DS-MoE layer (test and benchmark infrastructure).

This module only draws numbers and lays them out; it holds none of the layer's
arithmetic.  Both the CPU oracle's tests and the CUDA path's harness read their
inputs from here, so the two sides always see identical arrays.

Streams are counter-based (splitmix64 -> Box-Muller, implemented in ``gen.c``):
a tensor is identified by ``(seed, name)`` and element ``i`` depends on nothing
else, so any tensor can be regenerated anywhere, in any order.

bf16 tensors are returned as ``uint16`` bit patterns (rounded once, to nearest
even, from the fp32 draw); ``bf16_to_f32`` widens them exactly.
"""
from __future__ import annotations

import ctypes
import json
import math
import os
import subprocess
from dataclasses import dataclass, field, asdict

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libdsmoe_gen.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``gen.c`` with gcc into a shared object beside it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"]
        )
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64, dbl, vp = ctypes.c_uint64, ctypes.c_double, ctypes.c_void_p
        lib.dsmoe_gen_key.restype = u64
        lib.dsmoe_gen_key.argtypes = [u64, ctypes.c_char_p]
        for fn in (lib.dsmoe_gen_normal_f32, lib.dsmoe_gen_normal_bf16):
            fn.restype = None
            fn.argtypes = [u64, u64, u64, dbl, vp]
        lib.dsmoe_gen_uniform_f64.restype = None
        lib.dsmoe_gen_uniform_f64.argtypes = [u64, u64, u64, vp]
        lib.dsmoe_bf16_to_f32.restype = None
        lib.dsmoe_bf16_to_f32.argtypes = [vp, u64, vp]
        lib.dsmoe_f32_to_bf16.restype = None
        lib.dsmoe_f32_to_bf16.argtypes = [vp, u64, vp]
        _lib = lib
    return _lib


def key(seed: int, name: str) -> int:
    return int(_load().dsmoe_gen_key(seed, name.encode()))


def normal(seed: int, name: str, shape, scale: float = 1.0, dtype: str = "f32",
           first: int = 0) -> np.ndarray:
    """``scale * N(0,1)`` draws of stream ``(seed, name)``, elements ``first ..``.

    ``dtype='f32'`` gives float32; ``dtype='bf16'`` gives uint16 bf16 bit patterns.
    """
    lib = _load()
    shape = tuple(int(s) for s in (shape if hasattr(shape, "__len__") else (shape,)))
    n = int(np.prod(shape, dtype=np.int64)) if len(shape) else 1
    k = key(seed, name)
    if dtype == "f32":
        out = np.empty(n, dtype=np.float32)
        lib.dsmoe_gen_normal_f32(k, first, n, float(scale), out.ctypes.data)
    elif dtype == "bf16":
        out = np.empty(n, dtype=np.uint16)
        lib.dsmoe_gen_normal_bf16(k, first, n, float(scale), out.ctypes.data)
    else:
        raise ValueError(dtype)
    return out.reshape(shape)


def uniform(seed: int, name: str, n: int) -> np.ndarray:
    out = np.empty(int(n), dtype=np.float64)
    _load().dsmoe_gen_uniform_f64(key(seed, name), 0, int(n), out.ctypes.data)
    return out


def permutation(seed: int, name: str, n: int) -> np.ndarray:
    """A seeded permutation of ``range(n)`` (argsort of uniform draws)."""
    return np.argsort(uniform(seed, name, n), kind="stable").astype(np.int64)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float32)
    _load().dsmoe_bf16_to_f32(bits.ctypes.data, bits.size, out.ctypes.data)
    return out


def f32_to_bf16(vals: np.ndarray) -> np.ndarray:
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    out = np.empty(vals.shape, dtype=np.uint16)
    _load().dsmoe_f32_to_bf16(vals.ctypes.data, vals.size, out.ctypes.data)
    return out


def as_f32(a: np.ndarray) -> np.ndarray:
    """Widen a generated tensor (float32 or bf16 bits) to float32 values."""
    return bf16_to_f32(a) if a.dtype == np.uint16 else np.asarray(a, dtype=np.float32)


# --------------------------------------------------------------------------
# Workload recipes
# --------------------------------------------------------------------------

MODE_THRESHOLD, MODE_TOPK, MODE_ALL, MODE_THRESHOLD_TOPK = 0, 1, 2, 3


@dataclass
class LayerSpec:
    """Shape and selection rule of one MoE layer call (mirrors ``dsmoe_layer_desc``)."""
    name: str
    T: int
    d: int
    H: int
    E: int
    dtype: str = "bf16"            # storage type of x, W1, W2, out: 'f32' or 'bf16'
    mode: int = MODE_THRESHOLD
    eps: float = 0.0
    eps_normalized: int = 0
    K: int = 0
    min_k: int = 0
    out_fp32: int = 0
    fuse_combine: int = 0
    router_gain: float = 1.0       # scalar applied to the drawn Wr
    zipf_s: float = 0.0            # > 0: router bias b[e] = ln p, p ~ Zipf(s) over a seeded permutation
    seed: int = 0
    w2_gain: float = 1.0           # scalar applied to the drawn W2 (layer stacks: keeps the activations' scale)

    def replace(self, **kw) -> "LayerSpec":
        d = asdict(self)
        d.update(kw)
        return LayerSpec(**d)


def _calibration() -> dict:
    path = os.path.join(_HERE, "calibration.json")
    with open(path) as f:
        return json.load(f)


def spec(config: str, **overrides) -> LayerSpec:
    """The five benchmark workloads, by short name.

    c1 tiny fp32 threshold layer; c2 decode-shaped bf16 threshold layer (pass T);
    c3 prefill-shaped bf16 top-K layer; c4 dense (all-expert) forward; c5 skewed
    router with a Zipf(1.1) bias and a raw-score threshold sweep (pass eps).
    """
    cal = _calibration()
    if config == "c1":
        s = LayerSpec("c1", T=64, d=256, H=512, E=8, dtype="f32", mode=MODE_THRESHOLD,
                      eps=0.1, router_gain=cal["c1_router_gain"])
    elif config == "c2":
        s = LayerSpec("c2", T=32, d=2048, H=1024, E=32, dtype="bf16", mode=MODE_THRESHOLD,
                      eps=cal["c2_eps"])
    elif config == "c3":
        s = LayerSpec("c3", T=8192, d=3072, H=1536, E=32, dtype="bf16", mode=MODE_TOPK, K=12)
    elif config == "c4":
        s = LayerSpec("c4", T=16384, d=2048, H=1024, E=32, dtype="bf16", mode=MODE_ALL)
    elif config == "c5":
        s = LayerSpec("c5", T=4096, d=4096, H=1408, E=64, dtype="bf16", mode=MODE_THRESHOLD,
                      eps=0.01, zipf_s=1.1)
    else:
        raise KeyError(config)
    return s.replace(**overrides) if overrides else s


def tokens(s: LayerSpec, batch: str = "x") -> np.ndarray:
    """x[T,d] ~ N(0,1) in the layer's storage type; ``batch`` names the sub-stream."""
    return normal(s.seed, f"{s.name}.{batch}", (s.T, s.d), 1.0, s.dtype)


def router(s: LayerSpec, layer: int = 0):
    """(Wr[d,E] fp32 ~ gain*N(0,0.02^2), br[E] fp32 or None)."""
    Wr = normal(s.seed, f"{s.name}.Wr.{layer}", (s.d, s.E), 0.02 * s.router_gain, "f32")
    br = None
    if s.zipf_s > 0:
        ranks = np.arange(1, s.E + 1, dtype=np.float64) ** (-s.zipf_s)
        p = ranks / ranks.sum()
        perm = permutation(s.seed, f"{s.name}.zipf_perm.{layer}", s.E)
        br = np.log(p[perm]).astype(np.float32)
    return Wr, br


def experts(s: LayerSpec, layer: int = 0):
    """(W1[E,d,H], W2[E,H,d]) ~ N(0,0.02^2) in the layer's storage type."""
    W1 = normal(s.seed, f"{s.name}.W1.{layer}", (s.E, s.d, s.H), 0.02, s.dtype)
    W2 = normal(s.seed, f"{s.name}.W2.{layer}", (s.E, s.H, s.d), 0.02 * s.w2_gain, s.dtype)
    return W1, W2


def sample_tokens(s: LayerSpec, n: int, name: str = "sample") -> np.ndarray:
    """``n`` distinct token indices, seeded, ascending."""
    n = min(int(n), s.T)
    return np.sort(permutation(s.seed, f"{s.name}.{name}", s.T)[:n])
