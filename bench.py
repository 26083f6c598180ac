"""Benchmark of the DS-MoE layer forward on B200: MoE-layer tokens/s plus the roofline fraction of
the dominant kernel, with the CPU oracle timed beside it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2_t32|c2_t1|c2_t8|c3|c4|c5]
                    [--impl ours|reference] [--no-extra]

A step is one dsmoe_layer_forward over one batch of synthetic tokens.  The decode-shaped workloads
cycle through several distinct sets of expert weights (> L2 in total) so that every step reads its
weights from HBM, as consecutive layers of a real model do; the prefill-shaped and dense workloads
touch far more than L2 per step by themselves.  One JSON line goes to stdout.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import dsmoe_inputs as gi  # noqa: E402

WORKLOADS = {
    "c2_t1": ("c2", dict(T=1)), "c2_t8": ("c2", dict(T=8)), "c2_t32": ("c2", dict(T=32)),
    "c3": ("c3", {}), "c4": ("c4", {}), "c5": ("c5", dict(eps=0.01)),
    # the paper's own DS-MoE-6B layer shape (Table tab:model_arch: width 4096, 32 experts of width 512), not part
    # of the default run: narrower experts than the benchmark configurations
    "paper6b_t32": ("c2", dict(T=32, d=4096, H=512)), "paper6b_topk6": ("c3", dict(T=8192, d=4096, H=512, K=6)),
}
NCU_TRAFFIC_BYTES = {"c2_t32": 272.7e6, "c3": 1017.6e6}
DEFAULT_STEPS = {"c2_t1": 1000, "c2_t8": 1000, "c2_t32": 1000, "c3": 100, "c4": 50, "c5": 50, "paper6b_t32": 1000,
                 "paper6b_topk6": 100}
METRIC = "moe_layer_tokens_per_s"


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


def run_workload(name: str, steps: int, warmup: int, dist=None, with_e2e=True, sampler_index=0):
    import torch
    import paper_2404_05567_b200 as dm

    def to_dev(a):
        if a is None:
            return None
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    def desc_of(s):
        return dm.make_desc(s.T, s.d, s.H, s.E, dm.BF16 if s.dtype == "bf16" else dm.F32, s.mode, s.eps,
                            s.eps_normalized, s.K, s.min_k, s.out_fp32)

    cfg, kw = WORKLOADS[name]
    s = gi.spec(cfg, **kw)
    desc = desc_of(s)
    P = peaks()
    decode = s.T <= 128
    n_layers = 8 if decode else 1          # 8 x 268 MB of packed weights > 126 MB of L2
    Wr, br = gi.router(s)
    Wr_d, br_d = to_dev(Wr), to_dev(br)
    packed = []
    for layer in range(n_layers):
        W1, W2 = gi.experts(s, layer)
        W1_d, W2_d = to_dev(W1), to_dev(W2)
        pk = torch.empty(dm.dsmoe_packed_size(desc), dtype=torch.uint8, device="cuda")
        dm.dsmoe_pack_weights(desc, W1_d, W2_d, pk)      # one-off, outside every timed region
        torch.cuda.synchronize()
        packed.append(pk)
        del W1_d, W2_d, W1, W2
    x = gi.tokens(s)
    x_d = to_dev(x)
    ws = torch.empty(dm.dsmoe_workspace_size(desc), dtype=torch.uint8, device="cuda")
    out = torch.empty((s.T, s.d), dtype=torch.bfloat16, device="cuda")
    mask = torch.zeros(s.T, dtype=torch.int64, device="cuda")
    counts = torch.zeros(64, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")

    def step(i, want=False):
        dm.dsmoe_layer_forward(desc, x_d, Wr_d, br_d, None, None, packed[i % n_layers], out,
                               mask if want else None, counts if want else None, ws, status)

    step(0, want=True)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    cnt = counts[:s.E].cpu().numpy()
    A = int(cnt.sum())
    n_act = int((cnt > 0).sum())

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timed region
    for i in range(max(warmup, 3)):
        step(i)
    sampler = ClockSampler(sampler_index)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.finish()
    value, ms_total, world = job_throughput(dist, ms_total, s.T * steps)

    # ---- per-launch time of the dominant kernel (the tcgen05 expert GEMM), CUDA events inside the library
    dm.dsmoe_timing_enable(True)
    n_timed = min(steps, 200)
    durs = []
    for i in range(n_timed):
        step(i)
        durs.append(dm.dsmoe_timing_last())
    dm.dsmoe_timing_enable(False)
    durs = np.array(durs)                        # [n_timed, timed launches per step]
    per_step_launches = durs.shape[1]
    launch_ms = float(durs.sum(axis=1).mean())   # time inside the dominant kernel per step
    if decode:
        # selected experts' weights (W1 and W2), each byte once, all inside one launch of small_layer_kernel
        algo = 2.0 * n_act * s.d * s.H * 2.0
        roof = dict(bound="hbm", achieved=algo / (launch_ms * 1e-3) / 1e9, peak=P["hbm"], unit="GB/s",
                    peak_source=P["source"] + " (copy bandwidth)", kernel="small_layer_kernel")
    else:
        algo = 4.0 * A * s.d * s.H             # both projections: two launches of umma_gemm_kernel per step
        roof = dict(bound="tensor", achieved=algo / (launch_ms * 1e-3) / 1e12, peak=P["tf_sustained"],
                    unit="TFLOP/s", peak_source=P["source"] + " (sustained bf16)", kernel="umma_gemm_kernel")
    roof["frac"] = roof["achieved"] / roof["peak"]
    # dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures
    # summarised under profiles/ (c3: mean of the up- and down-projection launches); null where no capture was taken
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(name)
    roof["launch_ms"] = launch_ms / per_step_launches
    roof["launch_ms_each"] = [float(v) for v in durs.mean(axis=0)]
    roof["launches_per_step"] = per_step_launches
    roof["algorithmic_per_launch"] = algo / per_step_launches
    # whole-step figure against the same roofline (what the layer as a whole achieves)
    step_s = ms_total * 1e-3 / steps
    roof["step_frac"] = ((algo / step_s / 1e9) if decode else (algo / step_s / 1e12)) / roof["peak"]

    res = dict(value=value, ms_per_step=ms_total / steps, clocks=clocks, roofline=roof, A=A, active_experts=n_act,
               launches_per_step=(1 if decode else (5 if s.mode == gi.MODE_ALL else 9)), spec=s)

    # ---- end to end through the host-buffer entry point
    if with_e2e:
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
        e2e_value, ms_e2e, _ = job_throughput(dist, ms_e2e, s.T * steps)
        nbytes = s.T * s.d * 2
        res["e2e"] = {"value": e2e_value, "unit": "tokens/s",
                      "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": nbytes}
    del packed, ws
    torch.cuda.empty_cache()
    return res


def workload_config(name, s):
    mode = {0: "threshold", 1: "topk", 2: "all"}[s.mode]
    return {"workload": name, "T": s.T, "d": s.d, "E": s.E, "H": s.H, "select": mode, "eps": s.eps, "K": s.K,
            "l2": "decode: 8 weight sets cycled (2.1 GB > L2); prefill/dense: > L2 touched per step",
            "weights": "packed once outside the timed region"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_t32", choices=sorted(WORKLOADS))
    ap.add_argument("--no-extra", action="store_true")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    args = ap.parse_args()
    name = args.workload
    steps = args.steps if args.steps is not None else DEFAULT_STEPS[name]
    warmup = args.warmup if args.warmup is not None else 20
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    cfg, kw = WORKLOADS[name]
    s = gi.spec(cfg, **kw)

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

    res = run_workload(name, steps, warmup, dist=dist, sampler_index=physical_gpu_index(local_rank))
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    s = res["spec"]
    line = {"metric": METRIC, "value": res["value"], "unit": "tokens/s", "n_gpus": world, "steps": steps,
            "warmup": max(warmup, 3), "ms_per_step": res["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(name, s),
            "clocks": res["clocks"], "e2e": res.get("e2e"), "gpu_launches": res["launches_per_step"] * steps,
            "roofline": res["roofline"], "assignments": res["A"], "active_experts": res["active_experts"]}
    if world == 1:
        cb = oracle_tokens_per_s(s, budget_s=args.cpu_budget)
        line["cpu_baseline"] = {"value": cb["value"], "unit": "tokens/s", "cores": cb["cores"], "kind": "oracle",
                                "sample": cb["sample"]}
        if not args.no_extra:
            also = []
            for other, k in (("c2_t1", 500), ("c2_t8", 500), ("c3", 30), ("c4", 15)):
                if other == name:
                    continue
                r = run_workload(other, k, 5, with_e2e=False, sampler_index=physical_gpu_index(local_rank))
                also.append({"workload": other, "value": r["value"], "unit": "tokens/s", "ms_per_step": r["ms_per_step"],
                             "steps": k, "roofline": r["roofline"], "clocks": r["clocks"], "assignments": r["A"],
                             "active_experts": r["active_experts"]})
            line["also"] = also
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
