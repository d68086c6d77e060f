#!/usr/bin/env python
"""Benchmark of the MoE verification layer (one "step" = one moev_verify call: router
top-k -> expert union/grouping -> grouped SwiGLU expert FFN -> weighted combine).

Default workload: the DeepSeek-V3.1-shaped FP8 layer at gamma = 64 with scattered routing
(H=7168, I=2048, 256 routed + 1 shared expert, top-8 sigmoid), four distinct layers' weights
(45 GB) rotated call by call so no weight byte can be an L2 hit.  Prints ONE JSON line.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                  [--workload NAME] [--sweep]

N > 1 (under torchrun) runs N independent replicas, one per GPU (the path has no exchange
step); value is the aggregate over replicas, time the max over ranks.
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
import torch  # noqa: E402

import synth  # noqa: E402

METRIC = "moe_verify_expert_weight_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0

# workload name -> (shape, gamma, routing, kwargs)
WORKLOADS = {
    "deepseek_fp8_g64_scattered": ("deepseek", 64, "scattered", {}),
    "deepseek_fp8_g64_clustered": ("deepseek", 64, "clustered", {}),
    "qwen_bf16_g16": ("qwen", 16, "iid", {}),
    "qwen_bf16_g32": ("qwen", 32, "iid", {}),
    "qwen_bf16_g64": ("qwen", 64, "iid", {}),
    "gptoss_mxfp4_g8": ("gptoss", 8, "iid", {}),
    "gptoss_mxfp4_g16": ("gptoss", 16, "iid", {}),
    "gptoss_mxfp4_g32": ("gptoss", 32, "iid", {}),
    "gptoss_mxfp4_g64": ("gptoss", 64, "iid", {}),
    "tiny_fp32_g8": ("tiny", 8, "iid", {}),
    # batched verification (B requests x gamma tree tokens in one call) and skewed routing
    "deepseek_fp8_b4g64_scattered": ("deepseek", 256, "scattered", {}),
    "deepseek_fp8_b8g64_scattered": ("deepseek", 512, "scattered", {}),
    "deepseek_fp8_b4g64_zipf": ("deepseek", 256, "zipf", {"alpha": 1.0}),
    "deepseek_fp8_b8g64_zipf": ("deepseek", 512, "zipf", {"alpha": 1.0}),
    # profiling-size cases (a few GB on the device, still far larger than L2): the DeepSeek-
    # and Qwen-shaped layers with 64 experts
    "deepseek_fp8_E64_g16_profile": ("deepseek", 16, "scattered", {"_E": 64}),
    "qwen_bf16_E64_g16_profile": ("qwen", 16, "iid", {"_E": 64}),
    # the two-phase schedule (many tokens per expert) at profiling size: 256 rows, skewed routing
    "deepseek_fp8_E64_b4g64_zipf_profile": ("deepseek", 256, "zipf", {"_E": 64, "alpha": 1.0}),
    # routing kernels at the full router shape (256 experts, gamma 64) with thin experts (0.7 GB)
    "deepseek_router_profile": ("deepseek", 64, "scattered", {"_I": 128}),
    "deepseek_router_g8_profile": ("deepseek", 8, "scattered", {"_I": 128}),
    # tree-sized calls (the paper's operating point: a handful of tokens, 8 - 32 unique experts)
    "deepseek_fp8_g8_u8": ("deepseek", 8, "exact", {"U": 8}),
    "deepseek_fp8_g4_u16": ("deepseek", 4, "exact", {"U": 16}),
    "deepseek_fp8_E64_g8_u16_profile": ("deepseek", 8, "exact", {"_E": 64, "U": 16}),
}
DEFAULT_WORKLOAD = "deepseek_fp8_g64_scattered"

# DRAM (read + write) bytes per algorithmic byte of the dominant kernel, from the committed ncu
# capture of a smaller case of the same kernel (profiles/grouped_ffn_tc_fp8_E64_g16.md:
# 2.430690 GB + 5.26 MB against 2.422802 GB); traffic grows in proportion to the experts
# streamed, so the full-size launch is scaled by the same ratio.  Absent = not captured.
NCU_TRAFFIC_RATIO = {("fp8_e4m3", "tcgen05"): (2.430690e9 + 5.261312e6) / 2.422801920e9,
                     # profiles/grouped_ffn_mx_gptoss_g64.md: 1.462642 GB + 6.70 MB against 1.454112 GB
                     ("mxfp4", "tcgen05"): (1.462642e9 + 6.703872e6) / 1.454112e9,
                     # profiles/grouped_ffn_tc_bf16_E64_g16.md: 2.115337 GB + 3.93 MB against 2.113929 GB
                     ("bf16", "tcgen05"): (2.115337e9 + 3.926784e6) / 2.113929216e9}

ROUTING = {"iid": synth.make_iid_routing, "scattered": synth.make_scattered_routing,
           "clustered": synth.make_clustered_routing, "exact": synth.make_exact_union_routing,
           "zipf": synth.make_zipf_routing}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                mask = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def start(self):
        if self.nv:
            self._thr = threading.Thread(target=self._run, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr:
            self._thr.join()
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def workload_shape(name: str) -> synth.Shape:
    base, _, _, kw = WORKLOADS[name]
    shape = synth.SHAPES[base]
    if "_E" in kw:
        shape = shape.scaled(E=kw["_E"])
    if "_I" in kw:
        shape = shape.scaled(I=kw["_I"])
    return shape


def build_workload(name: str, n_layers: int, device, rank: int = 0, weights=None):
    """Inputs of a workload: per rotated layer its expert weights (generated, or taken from
    ``weights`` when another workload of the same shape already made them), router and x."""
    base, gamma, routing, kw = WORKLOADS[name]
    shape = workload_shape(name)
    kw = {k: v for k, v in kw.items() if not k.startswith("_")}
    layers = []
    for l in range(n_layers):
        lid = rank * 1000 + l
        w = weights[l] if weights is not None else synth.make_expert_weights(shape, layer=lid, device=device)
        wr, x = ROUTING[routing](shape, gamma, layer=lid, device=device, **kw)
        layers.append({"weights": w, "router_w": wr, "x": x})
    return shape, gamma, layers


def pack_layers(moev, layers):
    packed = []
    for L in layers:
        d = {"router_w": L["router_w"]}
        d.update({k: t for k, t in L["weights"].items() if t is not None})
        packed.append((moev.binding.make_layer(d), d))
    return packed


def time_calls(v, packed, xs, outs, gamma, steps, warmup):
    """Per-call latency of moev_verify (layers rotated call by call): a CUDA-event pair around
    every call, then the same calls once more with the per-kernel event records on.  Returns
    (sorted latencies in us, per-kernel mean us)."""
    n = len(packed)
    for i in range(max(warmup, n)):
        v.verify(packed[i % n][0], xs[i % n], gamma, outs[i % n])
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for i, (e0, e1) in enumerate(evs):
        e0.record()
        v.verify(packed[i % n][0], xs[i % n], gamma, outs[i % n])
        e1.record()
    torch.cuda.synchronize()
    lat = sorted(a.elapsed_time(b) * 1e3 for a, b in evs)
    v.profile_enable(True)
    for i in range(steps):
        v.verify(packed[i % n][0], xs[i % n], gamma, outs[i % n])
    kern_us, _ = v.profile_read()
    v.profile_enable(False)
    # the expert kernel's working time inside calls as they really run (dependent launches on): device
    # time stamps of its CTAs, earliest release by the routing kernels to latest exit, one call at a time
    v.ffn_span_enable(True)
    spans = []
    for i in range(min(steps, 16)):
        v.verify(packed[i % n][0], xs[i % n], gamma, outs[i % n])
        spans.append(v.ffn_span_read())
    v.ffn_span_enable(False)
    kern_us = list(kern_us) + [float(np.mean(spans)) if spans else 0.0]
    v.status_sync()
    return lat, kern_us


def fit_line(pts):
    """Least-squares latency = a + b U over (U, latency) points; returns None with fewer than two."""
    if len(pts) < 2:
        return None
    u = np.array([p[0] for p in pts], dtype=np.float64)
    t = np.array([p[1] for p in pts], dtype=np.float64)
    b, a = np.polyfit(u, t, 1)
    r2 = 1.0 - ((t - (a + b * u)) ** 2).sum() / max(((t - t.mean()) ** 2).sum(), 1e-30)
    return {"a_us": float(a), "b_us_per_expert": float(b), "r2": float(r2)}


def time_chain(moev, name, dev, weights, steps, warmup):
    """Dependent layers (layer l + 1 verifies layer l's output): one moev_verify_chain call over the
    rotated layers against the same layers as separate moev_verify calls on the same inputs."""
    n_layers = len(weights)
    shape, gamma, layers = build_workload(name, n_layers, dev, weights=weights)
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, gamma, shape.wfmt,
                          shape.afmt, shape.score, moev.IMPL_AUTO, shape.routed_scale)
    v = moev.MoeVerifier(cfg)
    packed = pack_layers(moev, layers)
    Ls = [p[0] for p in packed]
    outs = [v.alloc_out(gamma, diagnostics=False) for _ in layers]
    x0 = layers[0]["x"]

    def separate():
        for l in range(n_layers):
            v.verify(Ls[l], x0 if l == 0 else outs[l - 1]["y"], gamma, outs[l])

    res = {}
    for rep in range(2):  # both variants twice, alternating; the faster pass of each counts
        for label, fn in (("chain", lambda: v.verify_chain(Ls, x0, gamma, outs)), ("separate", separate)):
            for _ in range(max(2, warmup // 2)):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                fn()
            e1.record()
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / (steps * n_layers)
            res[label] = min(us, res.get(label, us))
    v.status_sync()
    U = [int(o["n_active"].item()) for o in outs]
    v.close()
    return {"workload": name, "gamma": gamma, "layers_per_call": n_layers, "U": U,
            "us_per_layer_chain": res["chain"], "us_per_layer_separate_calls": res["separate"],
            "note": "moev_verify_chain: x of layer l + 1 = y of layer l (layer 0 as the workload defines it)"}


def run_config_entry(moev, name, dev, weights, steps, warmup, peak):
    """One entry of the bench line's ``configs`` array: a benchmark configuration timed call by
    call (median of ``steps``), with the FFN kernel's own time and the clocks seen."""
    n_layers = len(weights)
    shape, gamma, layers = build_workload(name, n_layers, dev, weights=weights)
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, gamma, shape.wfmt,
                          shape.afmt, shape.score, moev.IMPL_AUTO, shape.routed_scale)
    v = moev.MoeVerifier(cfg)
    Wb = moev.expert_bytes(cfg)
    packed = pack_layers(moev, layers)
    xs = [L["x"] for L in layers]
    outs = [v.alloc_out(gamma, diagnostics=False) for _ in layers]
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    lat, kern_us = time_calls(v, packed, xs, outs, gamma, steps, warmup)
    clocks = sampler.stop()
    U = [int(o["n_active"].item()) for o in outs]
    nbytes = (float(np.mean(U)) + shape.n_shared) * Wb
    med = float(np.mean(lat))  # the layers rotated differ in U: the mean goes with the mean bytes
    v.close()
    return {"workload": name, "gamma": gamma, "U": U, "latency_us": med, "latency_median_us": lat[len(lat) // 2],
            "latency_min_us": lat[0],
            "gbs": nbytes / med / 1e3, "frac_of_8TBps": nbytes / med / 1e3 / NOMINAL_HBM_GBS,
            "ffn_kernel_us": kern_us[3], "ffn_frac_of_measured": nbytes / kern_us[3] / 1e3 / peak,
            "ffn_span_us": kern_us[6], "ffn_span_frac_of_measured": (nbytes / kern_us[6] / 1e3 / peak) if kern_us[6] > 0 else None,
            "routing_us": kern_us[0] + kern_us[1] + kern_us[2], "calls": steps,
            "clocks": {"sm_mhz": clocks["sm_mhz"], "reasons": clocks["reasons"]}}


def run_sweep_cells(moev, dev, weights, gammas, unions, steps, warmup, peak, emit=None):
    """Unique-expert sweep at the DeepSeek FP8 shape: routing built so that the union is exactly U.
    Returns (cells, fits per gamma)."""
    shape = synth.SHAPES["deepseek"]
    n_layers = len(weights)
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, max(gammas), shape.wfmt,
                          shape.afmt, shape.score, moev.IMPL_AUTO, shape.routed_scale)
    v = moev.MoeVerifier(cfg)
    Wb = moev.expert_bytes(cfg)
    cells, fits = [], {}
    for gamma in gammas:
        pts = []
        for U in unions:
            cell = {"gamma": gamma, "U": U}
            if not synth.union_feasible(shape, gamma, U):
                cell["latency_us"] = "n/a"
            else:
                layers = []
                for l in range(n_layers):
                    wr, x = synth.make_exact_union_routing(shape, gamma, U, layer=l, device=dev)
                    layers.append({"weights": weights[l], "router_w": wr, "x": x})
                packed = pack_layers(moev, layers)
                xs = [L["x"] for L in layers]
                outs = [v.alloc_out(gamma, diagnostics=False) for _ in layers]
                lat, kern_us = time_calls(v, packed, xs, outs, gamma, steps, warmup)
                assert all(int(o["n_active"].item()) == U for o in outs)
                med = lat[len(lat) // 2]
                nbytes = (U + shape.n_shared) * Wb
                cell.update(latency_us=med, latency_min_us=lat[0], latency_p90_us=lat[int(0.9 * len(lat))],
                            ffn_kernel_us=kern_us[3], ffn_span_us=kern_us[6], routing_us=kern_us[0] + kern_us[1] + kern_us[2],
                            bytes=nbytes, gbs=nbytes / med / 1e3,
                            frac_of_8TBps=nbytes / med / 1e3 / NOMINAL_HBM_GBS,
                            frac_of_measured=nbytes / med / 1e3 / peak, roofline_us_8TBps=nbytes / 8e6)
                pts.append((U, med))
            cells.append(cell)
            if emit:
                emit(dict(cell, sweep="unique_experts"))
        f = fit_line(pts)
        if f:
            f["roofline_b_us_per_expert_8TBps"] = Wb / 8e6
            fits[str(gamma)] = f
    v.close()
    return cells, fits


def layers_that_fit(shape: synth.Shape, want: int = 4) -> int:
    per_layer = (shape.E + shape.n_shared) * shape.bytes_per_expert()
    free, _ = torch.cuda.mem_get_info()
    return max(1, min(want, int((free * 0.85) // per_layer)))


ACT_QUANT = 0  # --act-quant: FP8 activations with 1x128 scales in front of both expert GEMMs (a variant, not the headline)


def ocfg_of(shape):
    import oracle
    return oracle.Config(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, shape.wfmt,
                         shape.afmt, shape.score, shape.routed_scale, act_quant=ACT_QUANT)


def time_oracle_sample(shape, layer, gamma_sample: int, repeats: int = 1):
    """The CPU oracle, as it stands, on the first gamma_sample tokens of one layer's input
    with that layer's full weights.  Returns (GB/s of expert-weight bytes, seconds, U, cores)."""
    import oracle
    host = synth.layer_to_numpy(layer["router_w"], layer["weights"])
    xs = synth.to_numpy(layer["x"][:gamma_sample].contiguous())
    best, U = None, 0
    for _ in range(repeats):
        t0 = time.perf_counter()
        res = oracle.moe_verify(ocfg_of(shape), host, xs, gamma_sample)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
        U = res.n_active
    nbytes = (U + shape.n_shared) * shape.bytes_per_expert()
    return nbytes / best / 1e9, best, U, oracle.num_threads()


def run_reference(args):
    """--impl reference: the oracle on the host cores, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shape = workload_shape(args.workload)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    shape_, gamma, layers = build_workload(args.workload, 1, dev)
    import oracle
    host = synth.layer_to_numpy(layers[0]["router_w"], layers[0]["weights"])
    gs = 1  # one token per step: k routed experts + shared
    cfg = ocfg_of(shape)
    steps, warm = max(1, min(args.steps, 5)), max(0, min(args.warmup, 1))
    tot_b, tot_t = 0, 0.0
    for i in range(warm + steps):
        xs = synth.to_numpy(layers[0]["x"][i % gamma:i % gamma + gs].contiguous())
        t0 = time.perf_counter()
        res = oracle.moe_verify(cfg, host, xs, gs)
        dt = time.perf_counter() - t0
        if i >= warm:
            tot_t += dt
            tot_b += (res.n_active + shape.n_shared) * shape.bytes_per_expert()
    val = tot_b / tot_t / 1e9
    sample = f"{gs} token(s) of the workload per step, full layer weights, {steps} steps"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": 1e3 * tot_t / steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": args.workload, "gamma": gamma},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(),
                             "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def aggregate_over_ranks(dist, device, ms_total: float, e2e_ms: float, nbytes: float):
    """Whole-job figures for N replicas: max time over ranks, bytes summed over ranks."""
    if dist is None:
        return ms_total, e2e_ms, nbytes
    t = torch.tensor([ms_total, e2e_ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    b = torch.tensor([float(nbytes)], device=device, dtype=torch.float64)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(b[0])


def run_ours(args):
    import paper_2607_12696_b200 as moev
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    shape = workload_shape(args.workload)
    n_layers = layers_that_fit(shape, args.layers)
    shape, gamma, layers = build_workload(args.workload, n_layers, dev, rank)
    impl = {"auto": moev.IMPL_AUTO, "simt": moev.IMPL_SIMT, "tcgen05": moev.IMPL_TCGEN05}[args.kernels]
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, gamma, shape.wfmt,
                          shape.afmt, shape.score, impl, shape.routed_scale, act_quant=ACT_QUANT)
    v = moev.MoeVerifier(cfg)
    packed = pack_layers(moev, layers)
    outs = [v.alloc_out(gamma, diagnostics=False) for _ in layers]
    Wb = moev.expert_bytes(cfg)

    def step(i):
        l = i % n_layers
        v.verify(packed[l][0], layers[l]["x"], gamma, outs[l])

    for i in range(args.warmup):
        step(i)
    v.status_sync()
    U = [int(o["n_active"].item()) for o in outs]
    if args.warmup < n_layers:  # make sure every layer's U is known
        for l in range(n_layers):
            step(l)
        torch.cuda.synchronize()
        U = [int(o["n_active"].item()) for o in outs]
    bytes_step = [(u + shape.n_shared) * Wb for u in U]

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing (the number: no per-kernel event records, kernels overlap their
    # launch latencies through programmatic dependent launch)
    sampler = ClockSampler(local)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    v.status_sync()
    tot_bytes = sum(bytes_step[i % n_layers] for i in range(args.steps))
    # ---- the same steps again with CUDA events recorded between the kernels of every call:
    # per-kernel durations for the roofline of the dominant kernel
    v.profile_enable(True)
    for i in range(min(args.steps, 500)):
        step(i)
    kern_us, kern_calls = v.profile_read()
    v.profile_enable(False)

    # ---- the rotated layers as one pipelined call per n_layers steps (independent inputs): the
    # next layer's router fills the tail of the previous layer's expert kernel
    pipe_us = None
    if n_layers > 1:
        Ls, xs_, os_ = [p[0] for p in packed], [L["x"] for L in layers], outs
        for _ in range(2):
            v.verify_pipeline(Ls, xs_, gamma, os_)
        n_calls = max(1, args.steps // n_layers)
        pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        pe0.record()
        for _ in range(n_calls):
            v.verify_pipeline(Ls, xs_, gamma, os_)
        pe1.record()
        barrier()
        pipe_us = pe0.elapsed_time(pe1) * 1e3 / (n_calls * n_layers)
        v.status_sync()

    # ---- end to end through the host-buffer entry point
    xh = [L["x"].cpu().pin_memory() for L in layers]
    yh = [torch.empty_like(t).pin_memory() for t in xh]
    nh = torch.zeros(1, dtype=torch.int32).pin_memory()
    for i in range(min(3, args.warmup)):
        v.verify_host(packed[i % n_layers][0], xh[i % n_layers], gamma, yh[i % n_layers], nh)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        l = i % n_layers
        v.verify_host(packed[l][0], xh[l], gamma, yh[l], nh)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    act_b = 4 if shape.afmt == synth.ACT_FP32 else 2
    h2d, d2h = gamma * shape.H * act_b, gamma * shape.H * act_b + 4

    # ---- aggregate over replicas: max time, summed bytes
    ms_total, e2e_ms, all_bytes = aggregate_over_ranks(dist, dev, ms_total, e2e_s * 1e3, float(tot_bytes))

    if rank == 0:
        value = all_bytes / (ms_total * 1e-3) / 1e9
        peak, peak_src = measured_peaks()
        impl_name = {1: "simt", 2: "tcgen05"}[v.resolved_impl()]
        mean_bytes = tot_bytes / args.steps
        if impl_name == "simt":  # two kernels; the first (gate/up) streams 2/3 of the bytes
            k_name, k_bytes, k_us = "ffn_gateup_simt", mean_bytes * 2.0 / 3.0, kern_us[3]
        else:
            k_name = "grouped_ffn_mx_kernel" if shape.wfmt == synth.W_MXFP4 else "grouped_ffn_tc_kernel"
            k_bytes, k_us = mean_bytes, kern_us[3]
        achieved = k_bytes / (k_us * 1e-6) / 1e9 if k_us > 0 else None
        dtype_name = {0: "f32", 1: "bf16", 2: "fp8_e4m3", 3: "mxfp4"}[shape.wfmt]
        cpu = None
        if not args.no_cpu_baseline:
            n_cpu = args.cpu_tokens if args.cpu_tokens > 0 else gamma
            cv, cs, cu, cores = time_oracle_sample(shape, layers[0], n_cpu)
            cpu = {"value": cv, "unit": UNIT, "cores": cores, "kind": "oracle",
                   "sample": f"first {n_cpu} of the {gamma} tokens of layer 0 (U={cu}"
                             f"+{shape.n_shared} experts streamed), full layer weights, {cs:.2f} s"}
        # ---- the other benchmark configurations and the unique-expert sweep, one after another
        # (default workload on one GPU only; each entry is a median over event-timed calls)
        configs, sweep_cells, sweep_fit, chains = None, None, None, None
        if args.workload == DEFAULT_WORKLOAD and world == 1 and not args.no_configs and ACT_QUANT == 0:
            cs_, cw = args.config_steps, 5
            ds_w = [L["weights"] for L in layers]
            configs = [run_config_entry(moev, "deepseek_fp8_g64_scattered", dev, ds_w, cs_, cw, peak),
                       run_config_entry(moev, "deepseek_fp8_g64_clustered", dev, ds_w, cs_, cw, peak)]
            sweep_cells, sweep_fit = run_sweep_cells(moev, dev, ds_w, [1, 4, 8, 32], [8, 16, 32, 64, 128, 256],
                                                     max(20, cs_ // 2), cw, peak)
            chains = [time_chain(moev, "deepseek_fp8_g64_scattered", dev, ds_w, max(10, cs_ // 4), cw),
                      time_chain(moev, "deepseek_fp8_g4_u16", dev, ds_w, max(20, cs_ // 2), cw)]
            del ds_w, packed
            layers.clear()
            torch.cuda.empty_cache()
            for base, names in (("qwen", ["qwen_bf16_g16", "qwen_bf16_g32", "qwen_bf16_g64"]),
                                ("gptoss", ["gptoss_mxfp4_g8", "gptoss_mxfp4_g16", "gptoss_mxfp4_g32",
                                            "gptoss_mxfp4_g64"])):
                shp = synth.SHAPES[base]
                ws = [synth.make_expert_weights(shp, layer=l, device=dev) for l in range(layers_that_fit(shp, 4))]
                for nm in names:
                    configs.append(run_config_entry(moev, nm, dev, ws, cs_, cw, peak))
                del ws
                torch.cuda.empty_cache()
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "pipelined": (None if pipe_us is None else
                          {"us_per_layer": pipe_us, "layers_per_call": n_layers,
                           "gbs": mean_bytes / pipe_us / 1e3, "note": "moev_verify_pipeline, independent inputs per layer"}),
            "dtype": dtype_name,
            "data": "synthetic",
            "config": {"workload": args.workload, "gamma": gamma, "H": shape.H, "I": shape.I,
                       "E": shape.E, "top_k": shape.top_k, "n_shared": shape.n_shared,
                       "unique_experts_per_layer": U, "layers_rotated": n_layers,
                       "l2_policy": "weights of %d layers (%.1f GB) rotated per call, > L2" % (
                           n_layers, n_layers * (shape.E + shape.n_shared) * Wb / 1e9),
                       "bytes_per_expert": Wb, "kernels": impl_name, "parallelism": "replicas",
                       **({"act_quant": ACT_QUANT} if ACT_QUANT else {})},
            "latency_us": 1e3 * ms_total / args.steps,
            "frac_of_8TBps": value / world / NOMINAL_HBM_GBS,
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                         "frac": (achieved / peak) if achieved else None,
                         "traffic": (k_bytes * NCU_TRAFFIC_RATIO[(dtype_name, impl_name)]
                                     if (dtype_name, impl_name) in NCU_TRAFFIC_RATIO else None),
                         "kernel": k_name, "kernel_us": k_us, "kernel_bytes": k_bytes,
                         "launches_timed": kern_calls,
                         "per_kernel_us": {"router_partial": kern_us[0], "topk_refine": kern_us[1],
                                           "route_group": kern_us[2], "ffn_1": kern_us[3],
                                           "ffn_2": kern_us[4], "finalize": kern_us[5]},
                         "peak_source": peak_src + " (of %s)" % peak_src},
            "cpu_baseline": cpu,
            "e2e": {"value": all_bytes / (e2e_ms * 1e-3) / 1e9, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms / args.steps,
                    "note": "host x -> device, layer, y + n_active -> host each step; expert "
                            "weights are layer parameters and stay resident"},
            "gpu_launches": v.launches_per_call() * args.steps,
            "clocks": clocks,
        }
        if configs is not None:
            line["configs"] = configs
            line["sweep"] = sweep_cells
            line["sweep_fit"] = sweep_fit
            line["chain"] = chains
        print(json.dumps(line))
    v.close()
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def run_sweep(args):
    """Unique-expert sweep at the DeepSeek FP8 shape: routing built so that the union is exactly
    U, for gamma in {1, 4, 8, 32, 128}; 4 layers' weights rotated per call.  Prints one JSON line
    per cell plus a linear fit latency = a + b U per gamma (rank 0, one GPU)."""
    import paper_2607_12696_b200 as moev
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    shape = synth.SHAPES["deepseek"]
    n_layers = layers_that_fit(shape, args.layers)
    weights = [synth.make_expert_weights(shape, layer=l, device=dev) for l in range(n_layers)]
    peak, peak_src = measured_peaks()
    gammas = [int(g) for g in args.sweep_gammas.split(",")]
    cells, fits = run_sweep_cells(moev, dev, weights, gammas, [8, 16, 32, 64, 128, 256], args.steps,
                                  args.warmup, peak, emit=lambda c: print(json.dumps(c), flush=True))
    print(json.dumps({"sweep": "unique_experts", "fit_latency_us = a + b*U": fits,
                      "layers_rotated": n_layers, "peak_source": peak_src}))


def run_select_demo(args):
    """Closing the loop of the paper on this path: cost-aware draft selection (Algorithm 1) in
    front of the verification layer, against acceptance-only selection (the same kernel with
    empty footprints, i.e. ranking by cumulative draft probability).  A binary draft tree of
    depth 7 (255 nodes) with expert locality along paths; each node's predicted expert set is
    its true single-layer routing (the paper's oracle-expert-set setting); gamma = 64 nodes are
    selected and verified on the DeepSeek-V3.1-shaped FP8 layer.  Prints one JSON line."""
    import paper_2607_12696_b200 as moev
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    shape = synth.SHAPES["deepseek"]
    gamma, depth = 64, 7
    n_layers = layers_that_fit(shape, 2)
    weights = [synth.make_expert_weights(shape, layer=l, device=dev) for l in range(n_layers)]
    parent, P, pred = synth.make_draft_tree(1, shape.E, shape.top_k, depth=depth, branch=2, seed_tag="demo-tree",
                                            p_reuse=args.p_reuse)
    wr, x_all = synth.make_tree_verify_inputs(shape, parent, pred, device=dev)
    cfg = moev.MoevConfig(shape.H, shape.I, shape.E, shape.top_k, shape.n_shared, gamma, shape.wfmt,
                          shape.afmt, shape.score, moev.IMPL_AUTO, shape.routed_scale)
    v = moev.MoeVerifier(cfg)
    Wb = moev.expert_bytes(cfg)
    packed = []
    for l in range(n_layers):
        d = {"router_w": wr}
        d.update({k: t for k, t in weights[l].items() if t is not None})
        packed.append((moev.binding.make_layer(d), d))
    t_parent = torch.from_numpy(parent).to(dev)
    t_P = torch.from_numpy(P).to(dev)
    t_pred = torch.from_numpy(pred.view(np.int32)).to(dev)
    result = {"demo": "draft selection -> verification layer", "tree_nodes": int(len(parent)), "gamma": gamma,
              "p_reuse": args.p_reuse, "workload": "deepseek_fp8, oracle expert sets, 1 layer", "layers_rotated": n_layers}
    for name, bitmaps in (("acceptance_only", torch.zeros_like(t_pred)), ("cost_aware", t_pred)):
        out = None
        for _ in range(3):
            out = moev.select_drafts(t_parent, t_P, bitmaps, gamma, 1e-6, out=out)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            out = moev.select_drafts(t_parent, t_P, bitmaps, gamma, 1e-6, out=out)
        e1.record()
        sel = out[0]
        torch.cuda.synchronize()
        sel_us = e0.elapsed_time(e1) * 1e3 / 20
        idx = sel.long()
        x = x_all[idx].contiguous()
        outs = [v.alloc_out(gamma, diagnostics=False) for _ in range(n_layers)]
        for i in range(max(args.warmup, n_layers)):
            v.verify(packed[i % n_layers][0], x, gamma, outs[i % n_layers])
        torch.cuda.synchronize()
        U = int(outs[0]["n_active"].item())
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for i, (a, b) in enumerate(evs):
            a.record()
            v.verify(packed[i % n_layers][0], x, gamma, outs[i % n_layers])
            b.record()
        torch.cuda.synchronize()
        lat = sorted(a.elapsed_time(b) * 1e3 for a, b in evs)
        med = lat[len(lat) // 2]
        result[name] = {"active_experts": U, "verify_latency_us": med, "selection_us": sel_us,
                        "sum_draft_prob": float(t_P[idx].sum().item()),
                        "expert_bytes": (U + shape.n_shared) * Wb,
                        "gbs": (U + shape.n_shared) * Wb / med / 1e3}
    a, c = result["acceptance_only"], result["cost_aware"]
    result["active_expert_reduction"] = 1.0 - c["active_experts"] / a["active_experts"]
    result["verify_latency_ratio"] = c["verify_latency_us"] / a["verify_latency_us"]
    print(json.dumps(result))
    v.close()


def run_select_bench(args):
    """Timing of the draft-selection kernels alone (Algorithm 1): the single-CTA kernel (255-node
    tree, one layer's expert bitmaps) and the cooperative multi-CTA kernel (the same tree with
    bitmaps over a whole model's 58 layers x 256 experts).  Prints one JSON line."""
    import paper_2607_12696_b200 as moev
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    out = {"bench": "draft selection kernels", "gamma": 64}
    for label, n_layers in (("single_cta_1_layer", 1), ("grid_58_layers", 58)):
        parent, P, pred = synth.make_draft_tree(n_layers, 256, 8, depth=7, branch=2, seed_tag="select-bench")
        tp, tP = torch.from_numpy(parent).to(dev), torch.from_numpy(P).to(dev)
        tpred = torch.from_numpy(pred.view(np.int32)).to(dev)
        o = None
        for _ in range(max(3, args.warmup)):
            o = moev.select_drafts(tp, tP, tpred, 64, 1e-6, out=o)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_calls = max(3, min(args.steps, 50))
        e0.record()
        for _ in range(n_calls):
            o = moev.select_drafts(tp, tP, tpred, 64, 1e-6, out=o)
        e1.record()
        torch.cuda.synchronize()
        out[label] = {"nodes": int(len(parent)), "bitmap_words": int(pred.shape[1]),
                      "us_per_call": e0.elapsed_time(e1) * 1e3 / n_calls, "n_selected": int(o[3].item())}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=4)
    ap.add_argument("--kernels", default="auto", choices=["auto", "simt", "tcgen05"])
    ap.add_argument("--cpu-tokens", type=int, default=0, help="tokens of layer 0 the oracle is timed on (0 = all gamma)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--act-quant", type=int, default=0, choices=[0, 1, 2],
                    help="FP8 activations with 1x128 scales (1: binary32 scales, 2: power-of-two scales)")
    ap.add_argument("--sweep", action="store_true", help="unique-expert sweep (DeepSeek FP8 shape) instead of the bench line")
    ap.add_argument("--sweep-gammas", default="1,4,8,32,128")
    ap.add_argument("--no-configs", action="store_true",
                    help="default workload only: skip the other configurations and the sweep behind the headline")
    ap.add_argument("--config-steps", type=int, default=50, help="timed calls per entry of the configs array")
    ap.add_argument("--select-demo", action="store_true",
                    help="cost-aware vs acceptance-only draft selection in front of the verification layer")
    ap.add_argument("--select-bench", action="store_true", help="time the draft-selection kernels alone")
    ap.add_argument("--p-reuse", type=float, default=0.7, help="expert locality along a tree path (select demo)")
    args = ap.parse_args()
    global ACT_QUANT
    ACT_QUANT = args.act_quant
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
        if args.sweep:
            run_sweep(args)
        elif args.select_demo:
            run_select_demo(args)
        elif args.select_bench:
            run_select_bench(args)
        else:
            run_ours(args)


if __name__ == "__main__":
    main()
