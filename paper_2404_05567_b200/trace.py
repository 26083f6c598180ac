"""Phase timeline of the decode kernel (a developer's diagnostic).

    python -m paper_2404_05567_b200.trace [--T 1] [--d 2048] [--H 1024] [--E 32] [--eps 0.03] [--reps 20]

Builds the library once more with -DDSMOE_TRACE into ``libdsmoe_trace.so`` (the kernels then record
``globaltimer`` stamps of their milestones per CTA), runs one decode-shaped layer a few times on random
inputs, and prints, per milestone, the median / minimum / maximum over the CTAs of the time since the
first CTA started, in microseconds.  Nothing here is part of the product path.
"""
from __future__ import annotations

import argparse
import ctypes
import glob
import os
import subprocess

import numpy as np
import torch

from . import binding
from .build import CSRC, NVCC_FLAGS, PKG, ROOT, _nvcc

SMALL_NAMES = {0: "CTA starts", 12: "router: first loads", 13: "router: slice sums done", 1: "router: at grid barrier",
               14: "router: grid barrier passed", 2: "router: partition known", 4: "MMA issuer: first tile in shared memory",
               3: "producer: up-projection issued", 28: "epilogue: first accumulator complete", 7: "epilogue: hg written, at grid barrier",
               5: "producer: down-projection weights prefetched", 6: "producer: grid barrier passed", 8: "MMA issuer: first down-projection tile",
               9: "epilogue: partial sums written", 10: "last grid barrier passed", 11: "CTA ends"}


def build_trace_lib() -> str:
    out = os.path.join(PKG, "libdsmoe_trace.so")
    objdir = os.path.join(ROOT, "_build", "trace")
    os.makedirs(objdir, exist_ok=True)
    objs = []
    for src in sorted(glob.glob(os.path.join(CSRC, "*.cu"))):
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        subprocess.check_call([_nvcc(), *NVCC_FLAGS, "-DDSMOE_TRACE", *os.environ.get("DSMOE_NVCC_EXTRA", "").split(),
                               "-c", src, "-o", obj])
        objs.append(obj)
    subprocess.check_call([_nvcc(), "-shared", "-o", out, *objs, "-Xcompiler", "-fPIC"])
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--T", type=int, default=1)
    ap.add_argument("--d", type=int, default=2048)
    ap.add_argument("--H", type=int, default=1024)
    ap.add_argument("--E", type=int, default=32)
    ap.add_argument("--eps", type=float, default=0.03)
    ap.add_argument("--topk", type=int, default=0, help="select exactly this many experts per token instead of the threshold")
    ap.add_argument("--reps", type=int, default=20)
    a = ap.parse_args()
    binding.LIB_PATH = build_trace_lib()
    binding._lib = None
    dm = binding
    torch.manual_seed(0)
    desc = (dm.make_desc(a.T, a.d, a.H, a.E, dm.BF16, dm.SELECT_TOPK, K=a.topk) if a.topk
            else dm.make_desc(a.T, a.d, a.H, a.E, dm.BF16, dm.SELECT_THRESHOLD, eps=a.eps))
    x = torch.randn(a.T, a.d, device="cuda").bfloat16()
    Wr = torch.randn(a.d, a.E, device="cuda") * 0.02
    layers = []
    for _ in range(8):
        W1 = (torch.randn(a.E, a.d, a.H, device="cuda") * 0.02).bfloat16()
        W2 = (torch.randn(a.E, a.H, a.d, device="cuda") * 0.02).bfloat16()
        pk = torch.empty(dm.dsmoe_packed_size(desc), dtype=torch.uint8, device="cuda")
        dm.dsmoe_pack_weights(desc, W1, W2, pk)
        layers.append(pk)
    ws = torch.empty(dm.dsmoe_workspace_size_packed(desc), dtype=torch.uint8, device="cuda")
    out = torch.empty(a.T, a.d, dtype=torch.bfloat16, device="cuda")
    counts = torch.zeros(64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for i in range(a.reps):
        dm.dsmoe_layer_forward(desc, x, Wr, None, None, None, layers[i % 8], out, None, counts, ws, status)
    torch.cuda.synchronize()
    print(f"T={a.T} d={a.d} H={a.H} E={a.E}: {int((counts[:a.E] > 0).sum())} experts selected, device status {int(status.item())}")
    L = dm.lib()
    buf = (ctypes.c_ulonglong * (192 * 32))()
    for reader, names in (("dsmoe_trace_read", SMALL_NAMES),):
        if not hasattr(L, reader) or getattr(L, reader)(buf) != 0:
            continue
        tr = np.frombuffer(buf, dtype=np.uint64).reshape(192, 32).astype(np.int64)
        live = tr[:, 0] > 0
        if not live.any():
            continue
        t0 = tr[live, 0].min()
        print(f"-- small_layer_kernel, last launch, {int(live.sum())} CTAs; microseconds after the first CTA's start: median / min / max")
        for idx, name in names.items():
            col = tr[live, idx]
            col = col[col > 0]
            if len(col):
                v = (col - t0) / 1e3
                print(f"{name:52s} {np.median(v):8.2f} {v.min():8.2f} {v.max():8.2f}   ({len(col)} CTAs)")


if __name__ == "__main__":
    main()
