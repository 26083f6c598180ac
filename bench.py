"""Benchmark of the DS-MoE layer forward on B200: MoE-layer tokens/s plus the roofline fraction of
the dominant kernel, with the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference] [--no-extra]

A step is one dsmoe_layer_forward over one batch of synthetic tokens.  The decode-shaped workloads
cycle through many distinct sets of expert weights (far more than L2 in total) so that every step reads
its weights from HBM, as consecutive layers of a real model do; the prefill-shaped and dense workloads
touch far more than L2 per step by themselves.  One JSON line goes to stdout.

--gpus N > 1 without a torchrun environment starts N ranks itself (one process per GPU); under
torchrun the ranks are already there.  The layer shards by token with no exchange, so the ranks are
replicas and the only collective is the reduction of the timing.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import dsmoe_inputs as gi  # noqa: E402

# name -> (recipe, overrides).  c1..c5 are the benchmark configurations; paper_* are the layer shapes of the paper's
# own models (Table tab:model_arch: DS-MoE-1B/3B/6B; Table tab:scaled: DS-MoE-10B/14B/19B), 32 experts each, top-K as
# the paper's speed tests use it (Table tab:latency: 6 for 3B, 4 for 6B; Table tab:scaled: 4).
PAPER_SHAPES = {"1b": (2048, 256, 6), "3b": (3072, 384, 6), "6b": (4096, 512, 4),
                "10b": (5120, 640, 4), "14b": (6144, 768, 4), "19b": (7168, 896, 4)}
WORKLOADS = {
    "c2_t1": ("c2", dict(T=1)), "c2_t8": ("c2", dict(T=8)), "c2_t32": ("c2", dict(T=32)),
    "c2_t64": ("c2", dict(T=64)), "c2_t128": ("c2", dict(T=128)), "c2_t256": ("c2", dict(T=256)), "c2_t512": ("c2", dict(T=512)),   # larger decode batches
    "c3": ("c3", {}), "c4": ("c4", {}),
    "c3_separate": ("c3", dict(fuse_combine=2)),   # aggregation as a second kernel instead of inside the down-projection (see dsmoe.h)
    "c5": ("c5", dict(eps=0.01)),
    # output-token throughput as the paper measures it ("GPU Inference Analysis"): a decode loop in which layer i's
    # output is layer i+1's input, 24 distinct layers (Table tab:model_arch: N_layer = 24 .. 36).  Between two layers
    # the activations are brought back to unit RMS by one elementwise multiply (a torch op standing in for the model's
    # normalisation layer, which is not part of this library), so that every layer's router sees inputs of the scale
    # the threshold was calibrated on
    "decode_loop_t8": ("c2", dict(T=8)), "decode_loop_t32": ("c2", dict(T=32)),
}
for _e in (0.0, 0.01, 0.05, 0.1, 0.2):
    WORKLOADS[f"c5_eps{_e}"] = ("c5", dict(eps=_e))
for _n, (_d, _H, _K) in PAPER_SHAPES.items():
    WORKLOADS[f"paper{_n}_prefill"] = ("c3", dict(T=8192, d=_d, H=_H, K=_K))
    WORKLOADS[f"paper{_n}_t32"] = ("c2", dict(T=32, d=_d, H=_H))
# dram bytes per launch of the dominant kernel from the ncu captures under profiles/ (c3: mean of the up- and down-projection)
NCU_TRAFFIC_BYTES = {"c2_t32": 273.3e6, "c3": 1529.6e6, "c4": 1910.0e6}
DEFAULT_STEPS = {"c3": 100, "c3_separate": 100, "c4": 50, "c4_backward": 20}
ALSO = [("c2_t1", 500), ("c2_t8", 500), ("c2_t128", 300), ("c3", 30), ("c3_separate", 30), ("c4", 15)] + [(f"c5_eps{e}", 15) for e in (0.0, 0.01, 0.05, 0.1, 0.2)] + \
       [(f"paper{n}_prefill", 30) for n in PAPER_SHAPES] + [(f"paper{n}_t32", 300) for n in ("1b", "3b", "6b", "19b")] + \
       [("decode_loop_t8", 20), ("decode_loop_t32", 20)]
METRIC = "moe_layer_tokens_per_s"
NOMINAL = dict(hbm=8000.0, tf=2250.0)     # datasheet: HBM3e GB/s, dense bf16 TFLOP/s
LOOP_LAYERS = 24


def default_steps(name):
    if name in DEFAULT_STEPS:
        return DEFAULT_STEPS[name]
    if name.startswith("decode_loop"):
        return 40                                   # x 24 layers per step
    if name.startswith("c5") or name.endswith("_prefill"):
        return 50
    return 1000


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), tf_burst=float(p["bf16_tflops"]),
                    tf_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def finish(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=1.0)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# --------------------------------------------------------------------------------------------
# CPU oracle legs (the only places this file may touch oracle/)
# --------------------------------------------------------------------------------------------

def oracle_tokens_per_s(s: gi.LayerSpec, budget_s: float, steps=None, warmup=0):
    """Times the oracle, as it stands, on a bounded token sample of the workload."""
    import oracle
    cores = oracle.num_threads()
    x = gi.tokens(s)
    Wr, br = gi.router(s)
    W1, W2 = gi.experts(s)
    S = oracle.router_scores(x, Wr, br)
    mask, k_t = oracle.select(S, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
    order = gi.sample_tokens(s, s.T, "cpu_sample")
    # one probe token per core to size the sample
    probe = order[:min(cores, s.T)]
    t0 = time.perf_counter()
    oracle.layer(x, W1, W2, S, mask, token_ids=probe)
    t_probe = max(time.perf_counter() - t0, 1e-4)
    if steps is None:
        n = int(min(s.T, max(len(probe), len(probe) * budget_s / t_probe)))
        ids = order[:n]
        xs = np.ascontiguousarray(x[ids])
        # small workloads finish in a fraction of a second: repeat the pass until about budget_s of CPU work
        reps = int(max(1, min(1000, budget_s / max(t_probe * n / len(probe), 1e-3))))
        t0 = time.perf_counter()
        for _ in range(reps):
            Ss = oracle.router_scores(xs, Wr, br)
            oracle.select(Ss, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
            oracle.layer(x, W1, W2, S, mask, token_ids=ids)
        dt = time.perf_counter() - t0
        return dict(value=n * reps / dt, cores=cores,
                    sample=f"{n} of {s.T} seeded tokens of {s.name}, {reps} passes, {dt:.1f} s",
                    ms_per_step=dt / reps * 1e3, steps=reps, n=n)
    # reference arm: every step is the same bounded sample
    total = steps + warmup
    n = int(min(s.T, max(1, (budget_s / total) / t_probe * len(probe))))
    n = max(n, min(cores, s.T))
    est = total * t_probe * max(1.0, n / len(probe))
    timed = steps
    if est > 1.5 * budget_s:
        timed = max(1, int(steps * budget_s / est))
    ids = order[:n]
    xs = np.ascontiguousarray(x[ids])

    def one():
        Ss = oracle.router_scores(xs, Wr, br)
        oracle.select(Ss, s.mode, s.eps, s.eps_normalized, s.K, s.min_k)
        oracle.layer(x, W1, W2, S, mask, token_ids=ids)

    for _ in range(min(warmup, 2)):
        one()
    t0 = time.perf_counter()
    for _ in range(timed):
        one()
    dt = time.perf_counter() - t0
    return dict(value=n * timed / dt, cores=cores,
                sample=f"{n} of {s.T} seeded tokens of {s.name} per step, {timed} steps timed", ms_per_step=dt / timed * 1e3,
                steps=timed, n=n)


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------

def job_throughput(dist, ms_local: float, tokens_local: int, device="cuda"):
    """Whole-job tokens/s of a token-sharded run: every rank processed `tokens_local` tokens of its own
    in `ms_local`; the job took as long as its slowest rank.  No data-path collective exists (each token's
    output depends on its own x and on replicated weights), only this reduction of the timing."""
    import torch
    if dist is None:
        return tokens_local / (ms_local * 1e-3), ms_local, 1
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([float(tokens_local)], dtype=torch.float64, device=device)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    ms = float(t.item())
    return float(n.item()) / (ms * 1e-3), ms, dist.get_world_size()


_PACKED = {}      # (d, H, E, recipe name, w2_gain, layer) -> packed weights on the device, shared between workloads


def packed_weights(dm, torch, s, desc, layer):
    key = (s.d, s.H, s.E, s.name, s.w2_gain, layer)
    if key not in _PACKED:
        W1, W2 = gi.experts(s, layer)
        W1_d = torch.from_numpy(W1.view(np.int16)).cuda().view(torch.bfloat16)
        W2_d = torch.from_numpy(W2.view(np.int16)).cuda().view(torch.bfloat16)
        pk = torch.empty(dm.dsmoe_packed_size(desc), dtype=torch.uint8, device="cuda")
        dm.dsmoe_pack_weights(desc, W1_d, W2_d, pk)      # one-off, outside every timed region
        torch.cuda.synchronize()
        _PACKED[key] = pk
    return _PACKED[key]


def drop_weights(torch, keep_shape=None):
    for k in list(_PACKED):
        if keep_shape is None or k[:3] != keep_shape:
            del _PACKED[k]
    torch.cuda.empty_cache()


def kernels_per_step(s, decode):
    """Launches of this library's kernels in one dsmoe_layer_forward (memsets are not kernels)."""
    if decode:
        return 1                                   # small_layer_kernel
    router = 3 if s.T > 256 else 1                 # split Wr, logits GEMM, softmax+select | one router kernel
    if s.mode == gi.MODE_ALL:
        return router + 2                          # up, down
    # chunk count, finalize, permute index, up, down, and the aggregation unless it runs inside the down-projection
    fused = s.fuse_combine == 1 or (s.fuse_combine == 0 and s.mode == gi.MODE_TOPK and s.H >= 1024 and
                                    s.T * min(s.K, s.E) >= 1024 * s.E)        # the library's rule (dsmoe.h)
    return router + 3 + 2 + (0 if fused else 1)


def run_workload(name: str, steps: int, warmup: int, dist=None, with_e2e=True, sampler_index=0, graph=False):
    import torch
    import paper_2404_05567_b200 as dm

    def to_dev(a):
        if a is None:
            return None
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    cfg, kw = WORKLOADS[name]
    s = gi.spec(cfg, **kw)
    desc = dm.make_desc(s.T, s.d, s.H, s.E, dm.BF16, s.mode, s.eps, s.eps_normalized, s.K, s.min_k, s.out_fp32,
                        s.fuse_combine)
    P = peaks()
    decode = s.T <= 128
    loop = name.startswith("decode_loop")
    # decode: distinct weight sets, at least 2 GB in all (L2 holds 126 MB), cycled; the loop workloads chain 24 of them
    per_layer = 4.0 * s.E * s.d * s.H
    n_layers = LOOP_LAYERS if loop else (max(3, min(8, int(np.ceil(2.1e9 / per_layer)))) if decode else 1)
    Wr, br = gi.router(s)
    Wr_d, br_d = to_dev(Wr), to_dev(br)
    packed = [packed_weights(dm, torch, s, desc, layer) for layer in range(n_layers)]
    x = gi.tokens(s)
    x_d = to_dev(x)
    ws = torch.empty(dm.dsmoe_workspace_size_packed(desc), dtype=torch.uint8, device="cuda")
    out = torch.empty((s.T, s.d), dtype=torch.bfloat16, device="cuda")
    act = [x_d, out, torch.empty_like(out)]           # loop workloads: layer i reads act[..] and writes the other
    mask = torch.zeros(s.T, dtype=torch.int64, device="cuda")
    counts = torch.zeros(64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def layer_call(i, src, dst, want=False):
        dm.dsmoe_layer_forward(desc, src, Wr_d, br_d, None, None, packed[i % n_layers], dst,
                               mask if want else None, counts if want else None, ws, status)

    scales = []                                   # loop workloads: 1 / RMS of each layer's output (set by the pre-pass)
    if loop:
        def step(i, want=False):
            # one decoding step of a 24-layer stack: x -> layer 0 -> layer 1 -> ... (each layer its own weights)
            src = x_d
            for layer in range(n_layers):
                dst = act[1 + layer % 2]
                layer_call(layer, src, dst, want and layer == 0)
                if scales:
                    dst.mul_(scales[layer])
                src = dst
    else:
        def step(i, want=False):
            layer_call(i, x_d, out, want)

    step(0, want=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    cnt = counts[:s.E].cpu().numpy()
    A = int(cnt.sum())
    n_act = int((cnt > 0).sum())
    n_act_layers, rms_layers = [n_act], []
    if loop:
        # what each layer of the stack really selects on the activations it gets (outside the timed region)
        n_act_layers, src = [], x_d
        for layer in range(n_layers):
            dst = act[1 + layer % 2]
            layer_call(layer, src, dst, True)
            torch.cuda.synchronize()
            n_act_layers.append(int((counts[:s.E] > 0).sum().item()))
            rms = dst.float().pow(2).mean().sqrt()
            rms_layers.append(float(rms.item()))
            scales.append((1.0 / rms).to(torch.bfloat16))
            dst.mul_(scales[-1])
            src = dst
    # selection statistics of this batch (stage calls, outside the timed region)
    scores = torch.empty((s.T, s.E), dtype=torch.float32, device="cuda")
    dm.dsmoe_router(desc, x_d, Wr_d, br_d, scores)
    st_d = torch.zeros(288, dtype=torch.uint8, device="cuda")
    dm.dsmoe_stats(desc, scores, mask, st_d)
    stats = dm.read_stats(st_d)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    calls_per_step = n_layers if loop else 1
    timed_per_call = 1 if decode else 2
    run_step = step
    if graph:
        # the whole step as one CUDA graph (launch overhead out of the way)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for i in range(3):
                step(i)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        # a graph holds as many consecutive steps as there are weight sets (they are cycled so that no step finds its
        # weights in L2), a second one the steps that remain: exactly `steps` steps are replayed
        per_graph = 1 if loop else n_layers
        graphs = {}
        for count in {per_graph, steps % per_graph} - {0}:
            graphs[count] = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graphs[count]):
                for i in range(count):
                    step(i)

        def run_step(i, want=False):
            if i % per_graph == 0:
                graphs[min(per_graph, steps - i)].replay()

    # ---- device-resident timed region.  The library's event pairs around the dominant kernel's launches cost a few
    # microseconds of stream time per step.  Prefill and dense steps (milliseconds) carry them in the timed loop itself:
    # the kernel times are then those of the very steps that give `value`.  Decode steps (tens of microseconds) are
    # timed clean, and the same un-synchronised loop runs once more with the event pairs for the kernel times.
    # warm-up: at least once through every weight set (they are cycled step by step), so that no timed step is the
    # first to touch its weights' pages
    for i in range(max(warmup, 3, 0 if loop else n_layers)):
        run_step(i)
    n_pairs = steps * calls_per_step * timed_per_call
    events_in_value_loop = n_pairs > 0 and not decode and not graph
    if events_in_value_loop:
        dm.dsmoe_timing_enable(n_pairs)
    sampler = ClockSampler(sampler_index)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        run_step(i)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.finish()
    value, ms_total, world = job_throughput(dist, ms_total, s.T * steps)
    durs, ms_evented = np.zeros(0), ms_total / steps
    if events_in_value_loop:
        durs = np.array(dm.dsmoe_timing_read(n_pairs))
        dm.dsmoe_timing_enable(0)
    elif n_pairs:
        dm.dsmoe_timing_enable(n_pairs)
        barrier()
        e0.record()
        for i in range(steps):
            step(i)                    # direct calls also where `value` came from graph replays: the events are the library's
        e1.record()
        barrier()
        ms_evented = e0.elapsed_time(e1) / steps
        durs = np.array(dm.dsmoe_timing_read(n_pairs))
        dm.dsmoe_timing_enable(0)
    assert int(status.item()) == 0

    step_s = ms_total * 1e-3 / steps
    res = dict(value=value, ms_per_step=ms_total / steps, clocks=clocks, A=A, active_experts=n_act, stats=stats,
               active_experts_per_layer=n_act_layers if loop else None, activation_rms_per_layer=rms_layers if loop else None,
               launches_per_step=kernels_per_step(s, decode) * calls_per_step, spec=s)
    if len(durs):
        durs = durs.reshape(steps, calls_per_step * timed_per_call)
        kernel_ms = float(durs.sum(axis=1).mean())        # time inside the dominant kernel per step
        capped = "sw_power_cap" in clocks["reasons"] or (clocks["sm_mhz"] and clocks["sm_max_mhz"] and
                                                          clocks["sm_mhz"] < 0.9 * clocks["sm_max_mhz"])
        weight_bytes = 2.0 * sum(n_act_layers) * s.d * s.H * 2.0 * (1 if loop else calls_per_step)
        flops = 4.0 * A * s.d * s.H * calls_per_step
        if decode:
            # selected experts' weights (W1 and W2), each byte once, all inside one launch of small_layer_kernel
            roof = dict(bound="hbm", achieved=weight_bytes / (kernel_ms * 1e-3) / 1e9, peak=P["hbm"], unit="GB/s",
                        peak_source=P["source"] + " (copy bandwidth)", kernel="small_layer_kernel")
            roof["frac"] = roof["achieved"] / roof["peak"]
            roof["frac_nominal"] = roof["achieved"] / NOMINAL["hbm"]
            roof["step_frac"] = weight_bytes / step_s / 1e9 / roof["peak"]
            roof["algorithmic_per_launch"] = weight_bytes / calls_per_step      # loop workloads: the mean over the layers
        else:
            # both projections: two launches of umma_gemm_kernel per step.  Peak: the burst figure unless the clock
            # samples of this very region show the power cap (then the sustained one applies)
            kind = "sustained" if capped else "burst"
            peak = P["tf_sustained"] if capped else P["tf_burst"]
            ach = flops / (kernel_ms * 1e-3) / 1e12
            roof = dict(bound="tensor", achieved=ach, peak=peak, unit="TFLOP/s",
                        peak_source=f"{P['source']} ({kind} bf16: clocks of this region {'show' if capped else 'show no'} power cap)",
                        kernel="umma_gemm_kernel", frac=ach / peak, frac_burst=ach / P["tf_burst"],
                        frac_sustained=ach / P["tf_sustained"], frac_nominal=ach / NOMINAL["tf"],
                        step_frac=flops / step_s / 1e12 / peak, algorithmic_per_launch=flops / 2)
            # where few assignments are left the weights' bytes bound the step, not the flops: the roofline time is
            # the larger of the two
            t_flop, t_byte = flops / (peak * 1e12), weight_bytes / (P["hbm"] * 1e9)
            roof["roofline_ms"] = max(t_flop, t_byte) * 1e3
            roof["roofline_bound"] = "tensor" if t_flop >= t_byte else "hbm"
            roof["frac_of_roofline_time"] = max(t_flop, t_byte) / (kernel_ms * 1e-3)
            roof["step_frac_of_roofline_time"] = max(t_flop, t_byte) / step_s
        # dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures
        # summarised under profiles/; null where no capture of the current kernel exists
        roof["traffic"] = NCU_TRAFFIC_BYTES.get(name)
        roof["kernel_ms_per_step"] = kernel_ms
        roof["ms_per_step_with_events"] = ms_evented     # the step time of the loop the kernel times were taken in
        roof["launch_ms_each"] = [float(v) for v in durs.mean(axis=0)[:timed_per_call]]
        roof["launches_per_step"] = calls_per_step * timed_per_call
        res["roofline"] = roof

    # ---- end to end through the host-buffer entry point
    if with_e2e and not loop:
        x_host = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory()
        out_host = torch.empty((s.T, s.d), dtype=torch.bfloat16).pin_memory()

        def step_host(i):
            dm.dsmoe_layer_forward_host(desc, x_host, x_d, Wr_d, br_d, None, None, packed[i % n_layers], out,
                                        out_host, ws, status)

        for i in range(3):
            step_host(i)
        barrier()
        e0.record()
        for i in range(steps):
            step_host(i)
        e1.record()
        barrier()
        ms_e2e = e0.elapsed_time(e1)
        serial_value, ms_e2e, _ = job_throughput(dist, ms_e2e, s.T * steps)
        # The calls as a serving loop would issue them (dsmoe_layer_forward_host_async: no wait inside the call): two
        # streams, each with its own device buffers, workspace and pinned output, steps alternating between them, so
        # that a step's copies run beside the other stream's kernel.  Every step still copies its input in and its
        # output out inside the timed region, which ends when both streams have drained.
        streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        sets = [(x_d, out, ws, status, out_host),
                (x_d.clone(), torch.empty_like(out), torch.empty_like(ws), torch.zeros_like(status),
                 torch.empty((s.T, s.d), dtype=torch.bfloat16).pin_memory())]

        def step_pipe(i):
            xd, o, w, st, oh = sets[i & 1]
            dm.dsmoe_layer_forward_host_async(desc, x_host, xd, Wr_d, br_d, None, None, packed[i % n_layers], o, oh, w, st,
                                              stream=streams[i & 1])

        torch.cuda.synchronize()
        for i in range(4):
            step_pipe(i)
        barrier()
        cur = torch.cuda.current_stream()
        e0.record(cur)
        for st in streams:
            st.wait_event(e0)
        t_issue = time.perf_counter()
        for i in range(steps):
            step_pipe(i)
        t_issue = (time.perf_counter() - t_issue) / steps * 1e3
        for st in streams:
            ev = torch.cuda.Event()
            ev.record(st)
            cur.wait_event(ev)
        e1.record(cur)
        barrier()
        for _, _, _, st, _ in sets:
            if int(st.item()) != 0:
                raise RuntimeError(f"device status {int(st.item())} in the end-to-end loop")
        e2e_value, ms_pipe, _ = job_throughput(dist, e0.elapsed_time(e1), s.T * steps)
        nbytes = s.T * s.d * 2
        res["e2e"] = {"value": max(e2e_value, serial_value), "unit": "tokens/s",
                      "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes,
                      "streams": 2 if e2e_value >= serial_value else 1, "one_stream_value": serial_value,
                      "two_stream_value": e2e_value, "host_issue_ms_per_step": t_issue}
    del packed, ws
    return res


# Mixture-of-attention-heads layer (Eq. 7-8) at DS-MoE-6B's attention shape (Table tab:model_arch: 8 experts of 4 heads
# of 128, model width 4096; 5 of 8 experts per token, the > 60 % layer utilisation the paper reports for attention):
# prefill = 32 sequences of 256 tokens (the sequence length of the paper's input-throughput setting), decode = one new
# token for each of 32 sequences with 2048 cached positions (its latency setting's context).
MOA_WORKLOADS = {
    "moa6b_prefill": dict(T=8192, d=4096, E=8, n_head=4, dh=128, K=5, n_seq=32, L=256, layout="prefill"),
    "moa6b_decode": dict(T=32, d=4096, E=8, n_head=4, dh=128, K=5, n_seq=32, L=2048, layout="decode"),
}


def run_moa(name: str, steps: int, warmup: int, sampler_index=0):
    import torch
    import paper_2404_05567_b200 as dm

    def to_dev(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    w = MOA_WORKLOADS[name]
    T, d, E, nh, dh, L, n_seq = w["T"], w["d"], w["E"], w["n_head"], w["dh"], w["L"], w["n_seq"]
    H = nh * dh
    s = gi.LayerSpec(name, T=T, d=d, H=H, E=E, dtype="bf16", mode=gi.MODE_TOPK, K=w["K"], router_gain=4.0)
    desc = dm.make_desc(T, d, H, E, dm.BF16, s.mode, 0.0, 0, s.K, 0, 0, 0)
    P = peaks()
    Wr, br = gi.router(s)
    Wq, Wo = gi.experts(s)
    packed = torch.empty(dm.dsmoe_packed_size(desc), dtype=torch.uint8, device="cuda")
    dm.dsmoe_pack_weights(desc, to_dev(Wq), to_dev(Wo), packed)
    # the key/value cache is drawn on the device (values of the same distribution as the generator's; no parity is
    # taken from this run): 32 x 4 x 2048 x 128 x 2 tensors would take the host generator a while
    g = torch.Generator(device="cuda").manual_seed(0)
    Kc = torch.randn((n_seq, nh, L, dh), generator=g, device="cuda").bfloat16()
    Vc = torch.randn((n_seq, nh, L, dh), generator=g, device="cuda").bfloat16()
    if w["layout"] == "prefill":
        per = T // n_seq
        seq = (np.arange(T) // per).astype(np.int32)
        pos = (np.arange(T) % per).astype(np.int32)
    else:
        seq = np.arange(T, dtype=np.int32)
        pos = np.full(T, L - 1, dtype=np.int32)
    seq_d, pos_d = to_dev(seq), to_dev(pos)
    x_d, Wr_d, br_d = to_dev(gi.tokens(s)), to_dev(Wr), to_dev(br) if br is not None else None
    ws = torch.empty(dm.dsmoe_workspace_size_packed(desc), dtype=torch.uint8, device="cuda")
    out = torch.empty((T, d), dtype=torch.bfloat16, device="cuda")
    counts = torch.zeros(64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    scale = 1.0 / float(np.sqrt(dh))

    def step(want=False):
        dm.dsmoe_moa_forward(desc, nh, scale, Kc, Vc, seq_d, pos_d, x_d, Wr_d, br_d, packed, out, None,
                             counts if want else None, ws, status)

    step(True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    A = int(counts[:E].sum().item())
    for _ in range(max(warmup, 3)):
        step()
    dm.dsmoe_timing_enable(3 * steps)
    sampler = ClockSampler(sampler_index)
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    clocks = sampler.finish()
    durs = np.array(dm.dsmoe_timing_read(3 * steps)).reshape(steps, 3).mean(axis=0)       # query projection, attention, output projection
    dm.dsmoe_timing_enable(0)
    assert int(status.item()) == 0
    proj_flops = 4.0 * A * d * H
    att_flops = 4.0 * w["K"] * nh * dh * float((pos.astype(np.float64) + 1).sum())
    kv_bytes = 2.0 * n_seq * nh * L * dh * 2 if w["layout"] == "decode" else 0.0
    weight_bytes = 2.0 * E * d * H * 2.0
    ach = proj_flops / ((durs[0] + durs[2]) * 1e-3) / 1e12
    t_flop, t_byte = (proj_flops + att_flops) / (P["tf_burst"] * 1e12), (weight_bytes + kv_bytes) / (P["hbm"] * 1e9)
    if t_flop >= t_byte:
        # many tokens: the two projections' flops against the measured GEMM rate (their two launches' time)
        head = dict(bound="tensor", achieved=ach, peak=P["tf_burst"], unit="TFLOP/s",
                    peak_source=P["source"] + " (burst bf16; the two projections)", frac=ach / P["tf_burst"],
                    frac_burst=ach / P["tf_burst"], frac_sustained=ach / P["tf_sustained"], frac_nominal=ach / NOMINAL["tf"])
    else:
        # few tokens: every expert's projection weights and the visible keys and values, read once, against the
        # measured copy bandwidth (all three launches' time)
        gbs = (weight_bytes + kv_bytes) / (float(durs.sum()) * 1e-3) / 1e9
        head = dict(bound="hbm", achieved=gbs, peak=P["hbm"], unit="GB/s", peak_source=P["source"] + " (copy bandwidth)",
                    frac=gbs / P["hbm"], frac_nominal=gbs / NOMINAL["hbm"])
    roof = dict(head, kernel="umma_gemm_kernel (projections) + moa_attention_mma_kernel", roofline_ms=max(t_flop, t_byte) * 1e3,
                frac_of_roofline_time=max(t_flop, t_byte) / (float(durs.sum()) * 1e-3),
                step_frac_of_roofline_time=max(t_flop, t_byte) / (ms * 1e-3), step_frac=max(t_flop, t_byte) / (ms * 1e-3),
                algorithmic_per_launch=proj_flops / 2, attention_flops=att_flops, kv_bytes=kv_bytes, traffic=None,
                kernel_ms_per_step=float(durs.sum()), ms_per_step_with_events=ms, launch_ms_each=[float(v) for v in durs],
                launches_per_step=3)
    return dict(workload=name, value=T / (ms * 1e-3), unit="tokens/s", ms_per_step=ms, steps=steps, roofline=roof, clocks=clocks,
                assignments=A, active_experts=E, config=dict(w))


def run_training_side(steps: int, warmup: int, sampler_index=0):
    """The training side of the layer at the dense forward's shape (C4): the gradients of dense training (Eq. 3) for a
    given output gradient -- two tensor-core launches, the recomputed activations and dO.W2^T with the gradients in its
    epilogue -- and the router's mutual-information loss with its gradient (Eq. 4-6)."""
    import torch
    import paper_2404_05567_b200 as dm

    def to_dev(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    s = gi.spec("c4")
    desc = dm.make_desc(s.T, s.d, s.H, s.E, dm.BF16, s.mode, s.eps, s.eps_normalized, s.K, s.min_k, 0, 0)
    P = peaks()
    Wr, br = gi.router(s)
    W1, W2 = gi.experts(s)
    W2_d = to_dev(W2)
    packed = packed_weights(dm, torch, s, desc, 0)
    x_d, Wr_d = to_dev(gi.tokens(s)), to_dev(Wr)
    br_d = to_dev(br) if br is not None else None
    scores = torch.empty((s.T, s.E), dtype=torch.float32, device="cuda")
    dm.dsmoe_router(desc, x_d, Wr_d, br_d, scores)
    g = torch.Generator(device="cuda").manual_seed(0)
    dO = torch.randn((s.T, s.d), generator=g, device="cuda").bfloat16()
    dS = torch.empty((s.T, s.E), dtype=torch.float32, device="cuda")
    dA = torch.empty((s.T, s.E * s.H), dtype=torch.bfloat16, device="cuda")
    loss3 = torch.zeros(3, dtype=torch.float32, device="cuda")
    grad = torch.empty((s.T, s.E), dtype=torch.float32, device="cuda")
    ws = torch.empty(dm.dsmoe_workspace_size_packed(desc), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def step():
        dm.dsmoe_dense_backward(desc, x_d, None, W2_d, packed, scores, None, dO, dS, dA, ws, status)

    for _ in range(max(warmup, 3)):
        step()
    dm.dsmoe_timing_enable(2 * steps)
    sampler = ClockSampler(sampler_index)
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    clocks = sampler.finish()
    durs = np.array(dm.dsmoe_timing_read(2 * steps)).reshape(steps, 2).mean(axis=0)
    dm.dsmoe_timing_enable(0)
    assert int(status.item()) == 0
    n_mi = 200
    for _ in range(5):
        dm.dsmoe_mi_loss(desc, scores, loss3, grad, ws)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n_mi):
        dm.dsmoe_mi_loss(desc, scores, loss3, grad, ws)
    e1.record()
    torch.cuda.synchronize()
    mi_us = e0.elapsed_time(e1) / n_mi * 1e3
    flops = 4.0 * s.T * s.E * s.d * s.H
    ach = flops / (float(durs.sum()) * 1e-3) / 1e12
    roof = dict(bound="tensor", kernel="umma_gemm_kernel", achieved=ach, peak=P["tf_burst"], unit="TFLOP/s",
                peak_source=P["source"] + " (burst bf16)", frac=ach / P["tf_burst"], frac_burst=ach / P["tf_burst"],
                frac_sustained=ach / P["tf_sustained"], frac_nominal=ach / NOMINAL["tf"],
                step_frac=flops / (ms * 1e-3) / 1e12 / P["tf_burst"], algorithmic_per_launch=flops / 2, traffic=None,
                kernel_ms_per_step=float(durs.sum()), ms_per_step_with_events=ms, launch_ms_each=[float(v) for v in durs],
                launches_per_step=2)
    return dict(workload="c4_backward", value=s.T / (ms * 1e-3), unit="tokens/s", ms_per_step=ms, steps=steps, roofline=roof,
                clocks=clocks, assignments=s.T * s.E, active_experts=s.E,
                mi_loss={"us_per_call": mi_us, "tokens": s.T, "experts": s.E, "with_gradient": True,
                         "bytes": 2.0 * s.T * s.E * 4, "L_MI": float(loss3[0].item())})


def workload_config(name, s):
    mode = {0: "threshold", 1: "topk", 2: "all", 3: "threshold_topk"}[s.mode]
    return {"workload": name, "T": s.T, "d": s.d, "E": s.E, "H": s.H, "select": mode, "eps": s.eps, "K": s.K,
            "l2": "decode: distinct weight sets cycled (>= 2 GB in all > L2; 24 chained in the loop workloads); prefill/dense: > L2 touched per step",
            "weights": "packed once outside the timed region"}


def free_port() -> int:
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def launch_ranks(n: int, argv) -> int:
    """Starts n copies of this script, one per GPU, with the rendezvous variables torchrun would set.
    Rank 0 inherits stdout (it prints the JSON line); the exit code is the worst of the ranks'."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + list(argv), env=env,
                                      stdout=None if r == 0 else subprocess.DEVNULL))
    rc = 0
    for p in procs:
        rc = max(rc, abs(p.wait()))
    return rc


def rendezvous_only(rank, world):
    """Everything of the N-rank run but the GPU work: process group (NCCL on GPUs, gloo without), barrier, and
    the reduction of a per-rank timing into the whole-job figure.  Used to check the launch path on CPU."""
    import torch
    import torch.distributed as td
    cuda = torch.cuda.is_available() and torch.cuda.device_count() >= world
    if cuda:
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    if world > 1:
        td.init_process_group("nccl" if cuda else "gloo")
        td.barrier()
    value, ms, n = job_throughput(td if world > 1 else None, 10.0 * (rank + 1), 1000, device="cuda" if cuda else "cpu")
    if rank == 0:
        print(json.dumps({"metric": METRIC, "rendezvous_only": True, "n_gpus": n, "value": value, "ms_per_step": ms,
                          "backend": "nccl" if cuda else "gloo"}))
    if world > 1:
        td.barrier()
        td.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_t32", choices=sorted(WORKLOADS) + sorted(MOA_WORKLOADS) + ["c4_backward"])
    ap.add_argument("--no-extra", action="store_true")
    ap.add_argument("--graph", action="store_true", help="replay each step as one CUDA graph")
    ap.add_argument("--fuse-combine", type=int, default=None, choices=[0, 1, 2],
                    help="override the workload's fuse_combine (see dsmoe.h)")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--rendezvous-only", action="store_true",
                    help="start the ranks, reduce a stand-in timing and print n_gpus; no GPU work")
    args = ap.parse_args()
    name = args.workload
    steps = args.steps if args.steps is not None else default_steps(name)
    warmup = args.warmup if args.warmup is not None else 20
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if name in MOA_WORKLOADS or name == "c4_backward":
        # the attention layer, or the training side, alone (one GPU; a diagnostic line: the default line is the
        # feed-forward layer's)
        import torch
        torch.cuda.set_device(0)
        from paper_2404_05567_b200 import build as lib_build
        lib_build.build()
        gi.build()
        r = run_training_side(steps, warmup) if name == "c4_backward" else run_moa(name, steps, warmup)
        print(json.dumps(dict(metric="dense_backward_tokens_per_s" if name == "c4_backward" else "moa_layer_tokens_per_s",
                              n_gpus=1, warmup=max(warmup, 3), higher_is_better=True, dtype="bf16", data="synthetic",
                              gpu_launches=(3 if name == "c4_backward" else 11) * steps, **r)))
        return
    if args.fuse_combine is not None:
        for k in WORKLOADS:
            WORKLOADS[k] = (WORKLOADS[k][0], dict(WORKLOADS[k][1], fuse_combine=args.fuse_combine))
    cfg, kw = WORKLOADS[name]
    s = gi.spec(cfg, **kw)

    if args.rendezvous_only:
        rendezvous_only(rank, world)
        return

    if args.impl == "reference":
        if rank != 0:
            return
        r = oracle_tokens_per_s(s, budget_s=150.0, steps=steps, warmup=warmup)
        line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "tokens/s", "n_gpus": args.gpus,
                "steps": r["steps"], "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                "config": workload_config(name, s),
                "cpu_baseline": {"value": r["value"], "unit": "tokens/s", "cores": r["cores"], "kind": "oracle",
                                 "sample": r["sample"]},
                "e2e": {"value": r["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    dist = None
    if world > 1:
        import torch.distributed as td
        torch.cuda.set_device(local_rank)
        td.init_process_group("nccl")
        dist = td
    else:
        torch.cuda.set_device(0)
    from paper_2404_05567_b200 import build as lib_build
    if rank == 0:
        lib_build.build()
        gi.build()
    if dist is not None:
        dist.barrier()

    res = run_workload(name, steps, warmup, dist=dist, sampler_index=physical_gpu_index(local_rank), graph=args.graph)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    s = res["spec"]
    st = res["stats"]
    line = {"metric": METRIC, "value": res["value"], "unit": "tokens/s", "n_gpus": world, "steps": steps,
            "warmup": max(warmup, 3), "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(name, s),
            "clocks": res["clocks"], "e2e": res.get("e2e"), "gpu_launches": res["launches_per_step"] * steps,
            "roofline": res.get("roofline"), "assignments": res["A"], "active_experts": res["active_experts"],
            "selection": {"near_threshold_1e-6": st["near_threshold"], "zero_tokens": st["zero_tokens"],
                          "empty_experts": st["empty_experts"]}}
    if world == 1:
        cb = oracle_tokens_per_s(s, budget_s=args.cpu_budget)
        line["cpu_baseline"] = {"value": cb["value"], "unit": "tokens/s", "cores": cb["cores"], "kind": "oracle",
                                "sample": cb["sample"]}
        if not args.no_extra:
            also = []
            shape = None
            for other, k in ALSO:
                if other == name:
                    continue
                so = gi.spec(WORKLOADS[other][0], **WORKLOADS[other][1])
                if shape is not None and (so.d, so.H, so.E) != shape:
                    drop_weights(torch, keep_shape=(so.d, so.H, so.E))   # keep the device's memory use bounded
                shape = (so.d, so.H, so.E)
                r = run_workload(other, k, 5, with_e2e=False, sampler_index=physical_gpu_index(local_rank))
                also.append({"workload": other, "value": r["value"], "unit": "tokens/s", "ms_per_step": r["ms_per_step"],
                             "steps": k, "roofline": r.get("roofline"), "clocks": r["clocks"], "assignments": r["A"],
                             "active_experts": r["active_experts"],
                             "active_experts_per_layer": r["active_experts_per_layer"],
                             "activation_rms_per_layer": r["activation_rms_per_layer"],
                             "near_threshold_1e-6": r["stats"]["near_threshold"]})
            drop_weights(torch)
            also.append(run_training_side(10, 3, sampler_index=physical_gpu_index(local_rank)))
            for other, k in (("moa6b_prefill", 20), ("moa6b_decode", 200)):
                drop_weights(torch)
                also.append(run_moa(other, k, 5, sampler_index=physical_gpu_index(local_rank)))
            line["also"] = also
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
