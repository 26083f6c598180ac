"""Where the kernels' time goes (a developer's diagnostic).

    python -m paper_2404_05567_b200.trace [--T 1] [--d 2048] [--H 1024] [--E 32] [--eps 0.03] [--reps 20]
    python -m paper_2404_05567_b200.trace --gemm prefill|dense [--fuse 0|1|2] [--pairs 0|1]

Builds the library once more with -DDSMOE_TRACE into ``libdsmoe_trace.so``.  Without ``--gemm``: the decode kernel
records ``globaltimer`` stamps of its milestones per CTA; one decode-shaped layer runs a few times on random inputs and
the tool prints, per milestone, the median / minimum / maximum over the CTAs of the time since the first CTA
started, in microseconds.  With ``--gemm``: the roles of the tensor-core GEMM kernel (MMA issuer, TMA producer, first
epilogue warp) count the clock cycles they spend waiting; a prefill-shaped (T=8192, d=3072, H=1536, top-K 12) or
dense-forward-shaped (T=16384, d=2048, H=1024, all 32 experts) layer runs a few times and the tool prints, per launch
of the layer, the median share of each role's time spent in each wait.  ``--pairs`` forces the kernel's form (single
CTAs / CTA pairs) instead of the library's own choice.  Nothing here is part of the product path.
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


def gemm_waits(a):
    if a.pairs is not None:
        os.environ["DSMOE_GEMM_PAIR"] = str(a.pairs)
    dm = binding
    torch.manual_seed(0)
    if a.gemm == "dense":
        T, d, H, E = 16384, 2048, 1024, 32
        desc = dm.make_desc(T, d, H, E, dm.BF16, dm.SELECT_ALL)
    elif a.gemm == "paper6b":      # the paper's 6B model: narrow experts, a short reduction in the down-projection
        T, d, H, E = 8192, 4096, 512, 32
        desc = dm.make_desc(T, d, H, E, dm.BF16, dm.SELECT_TOPK, K=4, fuse_combine=a.fuse)
    else:
        T, d, H, E = 8192, 3072, 1536, 32
        desc = dm.make_desc(T, d, H, E, dm.BF16, dm.SELECT_TOPK, K=12, fuse_combine=a.fuse)
    x = torch.randn(T, d, device="cuda").bfloat16()
    Wr = torch.randn(d, E, device="cuda") * 0.02
    W1 = (torch.randn(E, d, H, device="cuda") * 0.02).bfloat16()
    W2 = (torch.randn(E, H, d, device="cuda") * 0.02).bfloat16()
    pk = torch.empty(dm.dsmoe_packed_size(desc), dtype=torch.uint8, device="cuda")
    dm.dsmoe_pack_weights(desc, W1, W2, pk)
    ws = torch.empty(dm.dsmoe_workspace_size_packed(desc), dtype=torch.uint8, device="cuda")
    out = torch.empty(T, d, dtype=torch.bfloat16, device="cuda")
    counts = torch.zeros(64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(a.reps):
        dm.dsmoe_layer_forward(desc, x, Wr, None, None, None, pk, out, None, counts, ws, status)
    torch.cuda.synchronize()
    buf = (ctypes.c_longlong * (3 * 192 * 8))()
    if dm.lib().dsmoe_gemm_trace_read(buf) != 0:
        raise RuntimeError("dsmoe_gemm_trace_read failed")
    g = np.array(buf[:], dtype=np.float64).reshape(3, 192, 8)
    print(f"{a.gemm}: T={T} d={d} H={H} E={E}, pairs {'library' if a.pairs is None else a.pairs}, device status {int(status.item())}")
    print("-- umma_gemm_kernel, last launch of each kind; medians over the CTAs that hold the role")
    for k, name in enumerate(("router logits", "up-projection", "down-projection")):
        mm, pr, ep = g[k][g[k][:, 0] > 0], g[k][g[k][:, 3] > 0], g[k][g[k][:, 5] > 0]
        if not len(mm):
            continue
        print(f"{name:16s} MMA issuers {len(mm):3d}: {np.median(mm[:, 0]):9.0f} clk in all, {np.median(mm[:, 7]):4.0f} tiles; "
              f"waiting for operands {100 * np.median(mm[:, 1] / mm[:, 0]):5.1f} %, for a free accumulator {100 * np.median(mm[:, 2] / mm[:, 0]):5.1f} %"
              f" | producers {len(pr):3d}: waiting for a free slot {100 * np.median(pr[:, 4] / pr[:, 3]):5.1f} %"
              f" | epilogue warps: waiting for an accumulator {100 * np.median(ep[:, 6] / ep[:, 5]):5.1f} %")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--T", type=int, default=1)
    ap.add_argument("--d", type=int, default=2048)
    ap.add_argument("--H", type=int, default=1024)
    ap.add_argument("--E", type=int, default=32)
    ap.add_argument("--eps", type=float, default=0.03)
    ap.add_argument("--topk", type=int, default=0, help="select exactly this many experts per token instead of the threshold")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--gemm", choices=["prefill", "dense", "paper6b"], default=None, help="wait-time shares of the GEMM kernel's roles instead")
    ap.add_argument("--fuse", type=int, default=0, help="--gemm prefill: the layer's fuse_combine (0 library's choice, 1 inside, 2 separate)")
    ap.add_argument("--pairs", type=int, default=None, help="--gemm: 0 single CTAs, 1 CTA pairs wherever the shapes allow")
    a = ap.parse_args()
    binding.LIB_PATH = build_trace_lib()
    binding._lib = None
    if a.gemm:
        a.reps = min(a.reps, 5)
        return gemm_waits(a)
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
