"""Shared helpers of the GPU parity tests: move generated inputs to the device, call the C-ABI
through the binding, fetch results as numpy, and compare with the CPU oracle."""
from __future__ import annotations

import json
import os

import numpy as np
import torch

import dsmoe_inputs as gi
import oracle
import paper_2404_05567_b200 as dm

TOL_BF16 = 2e-2      # max|gpu - oracle| <= 2e-2 * RMS(oracle)   (bf16 storage, fp32 accumulate)
TOL_F32 = 1e-4       # max|gpu - oracle| <= 1e-4 * RMS(oracle)   (fp32)
NEAR = 1e-6          # scores this close to a decision boundary may legitimately flip


def record(kind: str, **fields):
    """Puts a measured figure on record: printed (pytest shows it with -s or on failure) and, when the
    environment variable DSMOE_PARITY_LOG names a file, appended there as one JSON line."""
    line = dict(kind=kind, **fields)
    print("[dsmoe]", json.dumps(line))
    path = os.environ.get("DSMOE_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(line) + "\n")


def to_dev(a: np.ndarray) -> torch.Tensor:
    """numpy (float32 / uint16 bf16 bits / ints) -> CUDA tensor with the matching torch dtype."""
    if a is None:
        return None
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
    if a.dtype == np.uint64:
        return torch.from_numpy(a.view(np.int64)).cuda()
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def np_f32(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy()


def desc_of(s: gi.LayerSpec) -> dm.LayerDesc:
    return dm.make_desc(s.T, s.d, s.H, s.E, dm.BF16 if s.dtype == "bf16" else dm.F32, s.mode, s.eps,
                        s.eps_normalized, s.K, s.min_k, s.out_fp32, s.fuse_combine)


def torch_dtype(s: gi.LayerSpec):
    return torch.bfloat16 if s.dtype == "bf16" else torch.float32


class Layer:
    """One synthetic layer resident on the GPU plus the numpy originals for the oracle."""

    def __init__(self, s: gi.LayerSpec, pack: bool = True, layer: int = 0, batch: str = "x"):
        self.s = s
        self.desc = desc_of(s)
        self.x = gi.tokens(s, batch)
        self.Wr, self.br = gi.router(s, layer)
        self.W1, self.W2 = gi.experts(s, layer)
        self.x_d, self.Wr_d, self.br_d = to_dev(self.x), to_dev(self.Wr), to_dev(self.br)
        self.W1_d, self.W2_d = to_dev(self.W1), to_dev(self.W2)
        self.packed = None
        if pack and s.dtype == "bf16" and s.d % 64 == 0 and s.H % 64 == 0:      # the packed layout is in blocks of 64
            self.packed = torch.empty(dm.dsmoe_packed_size(self.desc), dtype=torch.uint8, device="cuda")
            dm.dsmoe_pack_weights(self.desc, self.W1_d, self.W2_d, self.packed)
        # a call with packed weights needs only the tensor-core paths' (smaller) workspace
        nbytes = dm.dsmoe_workspace_size_packed(self.desc) if self.packed is not None else dm.dsmoe_workspace_size(self.desc)
        self.ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
        self.dev_status = torch.zeros(1, dtype=torch.int32, device="cuda")
        self.native = torch.float32 if s.dtype == "f32" else torch.bfloat16
        self.out = torch.empty((s.T, s.d), dtype=torch.float32 if s.out_fp32 else self.native, device="cuda")
        self.mask = torch.zeros(max(s.T, 1), dtype=torch.int64, device="cuda")
        self.counts = torch.zeros(64, dtype=torch.int32, device="cuda")

    def forward(self, want_counts: bool = True, out_fp32=None):
        """One dsmoe_layer_forward.  ``out_fp32`` overrides the spec's output type for this call."""
        desc, out = self.desc, self.out
        if out_fp32 is not None and int(out_fp32) != self.s.out_fp32:
            desc = desc_of(self.s.replace(out_fp32=int(out_fp32)))
            out = torch.empty((self.s.T, self.s.d), dtype=torch.float32 if out_fp32 else self.native, device="cuda")
        dm.dsmoe_layer_forward(desc, self.x_d, self.Wr_d, self.br_d, self.W1_d, self.W2_d, self.packed,
                               out, self.mask, self.counts if want_counts else None, self.ws, self.dev_status)
        torch.cuda.synchronize()
        assert int(self.dev_status.item()) == 0, f"device status {int(self.dev_status.item())}"
        return out

    # ---- oracle side
    def oracle_scores(self):
        return oracle.router_scores(self.x, self.Wr, self.br)

    def oracle_select(self, S):
        s = self.s
        return oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)


def check_mask_against_oracle(s: gi.LayerSpec, S: np.ndarray, mask_gpu: np.ndarray, mask_ref: np.ndarray):
    """The GPU decided on its own fp32 scores; any decision that differs from the oracle's must sit
    within NEAR of the boundary.  Returns (#flipped decisions, #scores within NEAR of the threshold)."""
    diff = mask_gpu ^ mask_ref
    flips = 0
    near = 0
    if s.mode in (gi.MODE_THRESHOLD, gi.MODE_THRESHOLD_TOPK):
        v = S * np.float32(s.E) if s.eps_normalized else S
        near = int((np.abs(v.astype(np.float64) - s.eps) <= NEAR).sum())
    # Threshold-TopK: one token's count flipping near the threshold may move the whole batch's K, so its tests use
    # inputs without such scores (near == 0); then K is the oracle's and only top-K ties may differ
    K = min(s.K, s.E)
    if s.mode == gi.MODE_THRESHOLD_TOPK:
        assert near == 0, "pick an eps that no score comes within 1e-6 of"
        K = bin(int(mask_ref[0])).count("1") if len(mask_ref) else 1
    for t in np.nonzero(diff)[0]:
        for e in range(s.E):
            if (int(diff[t]) >> e) & 1:
                flips += 1
                if s.mode == gi.MODE_THRESHOLD:
                    v = float(S[t, e]) * (s.E if s.eps_normalized else 1)
                    assert abs(v - s.eps) <= NEAR * (s.E if s.eps_normalized else 1), (t, e, v, s.eps)
                elif s.mode in (gi.MODE_TOPK, gi.MODE_THRESHOLD_TOPK):
                    kth = np.sort(S[t])[::-1][K - 1]
                    assert abs(float(S[t, e]) - float(kth)) <= NEAR, (t, e)
                else:
                    raise AssertionError("select-all cannot differ")
    return flips, near


def rel_err(gpu: np.ndarray, ref: np.ndarray) -> float:
    rms = float(np.sqrt(np.mean(ref.astype(np.float64) ** 2)))
    return float(np.max(np.abs(gpu.astype(np.float64) - ref))) / max(rms, 1e-300)


def rel_err_rows(gpu: np.ndarray, ref: np.ndarray) -> float:
    """Per-token form of the same bar: max_c |gpu[t,c] - ref[t,c]| / RMS(ref[t,:]), maximised over
    tokens.  Tokens are independent in Eq. 1, so this is the bar to use when row scales differ a lot
    (tokens that selected 1 expert next to tokens that selected 40).  Rows whose reference is all
    zero (no expert selected) must be exactly zero."""
    ref = ref.astype(np.float64)
    gpu = gpu.astype(np.float64)
    rms = np.sqrt(np.mean(ref ** 2, axis=1))
    zero = rms == 0
    assert np.all(gpu[zero] == 0.0)
    if np.all(zero):
        return 0.0
    e = np.max(np.abs(gpu[~zero] - ref[~zero]), axis=1) / rms[~zero]
    return float(e.max())


def layer_parity(s: gi.LayerSpec, pack: bool = True, sample: int | None = None):
    """Runs dsmoe_layer_forward and the oracle on the same inputs; returns a dict of measurements.

    ``sample`` = number of seeded tokens the oracle evaluates (None: all tokens)."""
    L = Layer(s, pack=pack)
    # The tolerance is applied to the value the layer computes, i.e. its fp32 output.  Storing that
    # value as bf16 is one more rounding (<= 2^-8 relative, by itself more than 2e-2 * RMS for any
    # element beyond 5.1 sigma), so the bf16 output is checked separately: it must be exactly the
    # round-to-nearest-even of the fp32 output.
    out_t = L.forward(out_fp32=True)
    out = out_t.cpu().numpy()
    if s.dtype == "bf16" and not s.out_fp32:
        out16 = L.forward(out_fp32=False)
        assert torch.equal(out16, out_t.to(torch.bfloat16)), "bf16 output is not RN(fp32 output)"
        L.out = out16
    else:
        L.out = out_t
    mask_gpu = to_np(L.mask)[:s.T].view(np.uint64)
    S = L.oracle_scores()
    mask_ref, k_ref = L.oracle_select(S)
    flips, near = check_mask_against_oracle(s, S, mask_gpu, mask_ref)
    counts_gpu = to_np(L.counts)[:s.E]
    counts_from_mask = np.array([int(((mask_gpu >> np.uint64(e)) & np.uint64(1)).sum()) for e in range(s.E)])
    assert np.array_equal(counts_gpu, counts_from_mask)
    ids = None if sample is None or sample >= s.T else gi.sample_tokens(s, sample)
    if ids is not None:
        # the compared tokens must reach every expert that any token selected: where the seeded sample misses
        # one, the first token that selected it joins the sample
        seen = np.bitwise_or.reduce(mask_gpu[ids]) if len(ids) else np.uint64(0)
        missing = int(np.bitwise_or.reduce(mask_gpu)) & ~int(seen)
        extra = [int(np.nonzero((mask_gpu >> np.uint64(e)) & np.uint64(1))[0][0]) for e in range(s.E) if (missing >> e) & 1]
        if extra:
            ids = np.unique(np.concatenate([ids, np.array(extra, dtype=ids.dtype)]))
    ref = oracle.layer(L.x, L.W1, L.W2, S, mask_gpu, token_ids=ids)
    got = out if ids is None else out[ids]
    # the tolerance is relative to the RMS of the oracle's output over the compared tokens
    err = rel_err(got, ref) if ref.size else 0.0
    err_rows = rel_err_rows(got, ref) if ref.size else 0.0
    record("layer_parity", name=s.name, T=s.T, d=s.d, H=s.H, E=s.E, dtype=s.dtype, mode=s.mode, eps=s.eps, K=s.K,
           packed=bool(L.packed is not None), tokens_compared=int(ref.shape[0]), err_global=err, err_per_token=err_rows,
           flips=flips, near_threshold=near, A=int(counts_gpu.sum()))
    return dict(err=err, err_rows=err_rows, flips=flips, near=near, A=int(counts_gpu.sum()), layer=L, ref=ref, got=got,
                empty_experts=int((counts_gpu == 0).sum()),
                zero_tokens=int((mask_gpu == 0).sum()))
