#!/usr/bin/env python
"""Benchmark of the dynamic-k MoE layer (D2DMoE inference hot path) on B200.

One step = one pass of the whole hot path (router_fwd -> select_dynk -> moe_ffn_fwd, the single
C-ABI call d2d_layer_fwd) over one batch of synthetic tokens.  Default workload: the largest
single-GPU configuration, the Llama-style gated layer (d=4096, d_ff=11008, 344 experts x 32
neurons, 8192 tokens) at tau = 0.4; the other configurations are timed in the same run and
reported in `per_config` of the same JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama] [--tau 0.4]
                    [--tokens T] [--bernoulli p] [--path auto|dense|gather|fused] [--experts-per-group g] [--fp8-experts]
                    [--sweep] [--no-per-config] [--no-cpu-baseline] [--no-graph] [--group N]
    python bench.py --impl reference ...      # times the CPU oracle on the host cores

Prints ONE JSON line on stdout (rank 0).  Multi-GPU: launched by torch.distributed.run, one
process per GPU, each rank runs the same layer on its own batch (tokens are independent: no
data-path collective), value = all ranks' tokens / max-over-ranks time ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "dynamic-k MoE layer tokens/s"
UNIT = "tokens/s"
L2_FLUSH_BYTES = 256 << 20

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from ncu captures of that
# kernel on that workload (absent: no capture of that combination); keyed by (workload, tokens, kernel).
# The full-size figures are one-pass captures of those two counters alone: the masked dense up projection reads
# 610.4 MB and writes 174.9 MB; the gathered one (tau = 0.4) reads 2911.9 MB and writes 107.8 MB (token rows and
# weight rows together exceed what L2 keeps, so rows are fetched again for many of the groups that use them).
NCU_TRAFFIC_BYTES = {
    ("llama", 8192, "dense_up"): 610_425_088 + 174_942_464,
    ("llama", 8192, "gather_up"): 2_911_860_736 + 107_819_520,
}

# (workload, tokens or None = the workload's own, tau or None, Bernoulli p or None) timed for `per_config`
PER_CONFIG = [
    ("tiny", None, 0.5, None),
    ("bert", None, 0.3, None), ("bert", None, 0.7, None),
    ("vit", None, 0.3, None), ("vit", None, 0.6, None),
    ("gpt2_ffn", 1, 0.5, None), ("gpt2_ffn", 8, 0.5, None), ("gpt2_ffn", 64, 0.5, None),
    ("gpt2_attn", 1, 0.5, None), ("gpt2_attn", 64, 0.5, None),
    ("llama", None, 0.6, None),
    # decode on the Llama shape, where the kept experts' bytes set the time: bf16 weights, then 8-bit (e4m3) weights
    ("llama", 1, 0.2, None), ("llama", 1, 0.2, None, True), ("llama", 2, 0.2, None), ("llama", 2, 0.2, None, True),
    ("paper", None, None, 0.02), ("paper", None, None, 0.05), ("paper", None, None, 0.1), ("paper", None, None, 0.3),
    ("paper", None, None, 0.5),
]


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=50)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="llama")
    p.add_argument("--tokens", type=int, default=0, help="override the workload's token count")
    p.add_argument("--tau", type=float, default=None, help="threshold of the dynamic-k rule (default 0.4)")
    p.add_argument("--bernoulli", type=float, default=None,
                   help="override the gating decisions with Bernoulli(p) samples (the latency protocol of Sec. 4.4): "
                        "the timed step is then the expert step d2d_moe_ffn_fwd on that mask")
    p.add_argument("--path", default="auto", choices=["auto", "dense", "gather", "fused"],
                   help="which up projection the tensor-core expert step uses (d2d_layer_set_expert_path)")
    p.add_argument("--experts-per-group", type=int, default=0, help="group size of the gathered path (0 = default)")
    p.add_argument("--fp8-experts", action="store_true",
                   help="expert weights as 8-bit e4m3 codes with one power-of-two scale per expert (d2d_layer_create_fp8)")
    p.add_argument("--sweep", action="store_true", help="also time the workload's whole tau grid")
    p.add_argument("--no-per-config", action="store_true", help="skip the other configurations")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a captured CUDA graph")
    p.add_argument("--group", type=int, default=0,
                   help="also time N layers of the workload's shape on the shared input as one d2d_group_fwd call "
                        "(the Q, K, V projections of an attention layer) against N separate d2d_layer_fwd calls")
    args = p.parse_args()
    if args.tau is None:
        args.tau = 0.4
    return args


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.001):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

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
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": (statistics.median(self.samples) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def config_dict(cfg, tau, bernoulli=None):
    """The workload as both arms name it (the same keys and values in `--impl ours` and `--impl reference`)."""
    c = {"workload": cfg.name, "tokens": cfg.T, "d": cfg.d, "d_ff": cfg.d_ff, "experts": cfg.E, "expert_size": cfg.s,
         "d_h": cfg.d_h, "act": cfg.act, "gated": cfg.gated, "tau": tau}
    if bernoulli is not None:
        c["tau"] = None
        c["bernoulli_p"] = bernoulli
    return c


def stats(ts):
    ts = sorted(ts)
    return {"mean": sum(ts) / len(ts), "median": ts[len(ts) // 2], "min": ts[0]}


# ------------------------------------------------------------------------------------------ CPU oracle arm

def oracle_step_fn(cfg, weights, x_sample, tau, G_sample=None):
    import oracle
    act = oracle.ACT_BY_NAME[cfg.act]
    if G_sample is not None:
        def step():
            return oracle.moe_ffn(x_sample, weights["w1"], weights["b1"], weights["w_gate"], weights["w2"], weights["b2"], act, G_sample)
        return step

    def step():
        return oracle.layer(x_sample, weights, act, tau)
    return step


def time_cpu_oracle(cfg, weights, x, tau, budget_s=12.0):
    """Times the oracle, as it stands, on a bounded token sample sized for roughly budget_s seconds."""
    import oracle
    probe = min(16, x.shape[0])
    t0 = time.perf_counter()
    oracle_step_fn(cfg, weights, x[:probe], tau)()
    per_tok = (time.perf_counter() - t0) / probe
    n = int(max(probe, min(x.shape[0], budget_s / max(per_tok, 1e-9))))
    passes = int(max(1, min(1000, budget_s / max(per_tok * n, 1e-9))))
    step = oracle_step_fn(cfg, weights, x[:n], tau)
    t0 = time.perf_counter()
    for _ in range(passes):
        step()
    dt = time.perf_counter() - t0
    threads = max(1, oracle.num_threads())
    n1 = max(1, min(n, int(3.0 / max(per_tok * threads, 1e-9))))       # about three seconds on one thread
    oracle.set_num_threads(1)
    t1 = time.perf_counter()
    oracle_step_fn(cfg, weights, x[:n1], tau)()
    dt1 = time.perf_counter() - t1
    oracle.set_num_threads(threads)
    return {"value": n * passes / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": f"first {n} of {x.shape[0]} tokens of the {cfg.name} workload at tau={tau}, {passes} passes "
                      f"(router+select+metadata+experts each), {dt:.2f} s",
            "single_thread_value": n1 / dt1, "single_thread_sample": f"first {n1} tokens, one pass, {dt1:.2f} s"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from paper_2310_04361_b200 import workloads as wl
    cfg = wl.CONFIGS[args.workload]
    if args.tokens:
        cfg = wl.with_tokens(cfg, args.tokens)
    weights = wl.make_weights(cfg)
    x = wl.make_tokens(cfg)
    G = wl.make_bernoulli_mask(cfg, args.bernoulli) if args.bernoulli is not None else None
    probe = min(8, cfg.T)
    t0 = time.perf_counter()
    oracle_step_fn(cfg, weights, x[:probe], args.tau, None if G is None else G[:probe])()
    per_tok = (time.perf_counter() - t0) / probe
    total_steps = args.steps + args.warmup
    n = int(max(1, min(cfg.T, 90.0 / total_steps / max(per_tok, 1e-9))))   # whole run within ~1.5 minutes
    step = oracle_step_fn(cfg, weights, x[:n], args.tau, None if G is None else G[:n])
    for _ in range(args.warmup):
        step()
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        step()
        times.append(time.perf_counter() - t0)
    dt = sum(times)
    value = n * args.steps / dt
    sample = f"each step = the first {n} of {cfg.T} tokens of the {cfg.name} workload"
    st = stats([1e3 * t for t in times])
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "ms_median": st["median"], "ms_min": st["min"],
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, args.tau, args.bernoulli),
        "tokens_per_step": n,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------ GPU arm

class Harness:
    """Timing protocol shared by every measurement of the GPU arm: W untimed warm-up steps, then K steps each
    bracketed by CUDA events on the launching stream, with an L2 flush (a 256 MiB write) before every step and
    outside its events; the step is a CUDA-graph replay of the library's own launch sequence unless --no-graph."""

    def __init__(self, torch, dev, dist, world, no_graph):
        self.torch, self.dev, self.dist, self.world, self.no_graph = torch, dev, dist, world, no_graph
        self.flush = torch.empty((L2_FLUSH_BYTES,), dtype=torch.uint8, device=dev)
        self.stream = torch.cuda.current_stream()
        self.all_ranks = True        # False for the measurements only rank 0 takes (no collective barrier then)

    def barrier(self):
        if self.world > 1 and self.all_ranks:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def timed_loop(self, fn, steps, warmup):
        torch = self.torch
        for _ in range(warmup):
            self.flush.zero_()
            fn()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        self.barrier()
        for a, b in evs:
            self.flush.zero_()
            a.record(self.stream)
            fn()
            b.record(self.stream)
        self.barrier()
        return [a.elapsed_time(b) for a, b in evs]       # ms

    def runner(self, fn):
        torch = self.torch
        if self.no_graph:
            return fn
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(3):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g.replay

    def time(self, fn, steps, warmup=3):
        return stats(self.timed_loop(self.runner(fn), steps, warmup))

    def time_interleaved(self, fns, steps, warmup=3):
        """Times several step functions in one round-robin loop (a, b, c, a, b, c, ...), each step with its own events
        and its own L2 flush: all of them see the same clock and power state.  A B200 runs a tensor-bound step about
        10 % faster for the first 0.2 s after an idle period than under sustained load (measured: 1.56 ms against
        1.73 ms for the Llama-shaped layer), so medians taken in separate loops are not comparable."""
        torch = self.torch
        runs = [self.runner(fn) for fn in fns]
        for _ in range(warmup):
            for r in runs:
                self.flush.zero_()
                r()
        evs = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)] for _ in runs]
        self.barrier()
        for i in range(steps):
            for j, r in enumerate(runs):
                a, b = evs[j][i]
                self.flush.zero_()
                a.record(self.stream)
                r()
                b.record(self.stream)
        self.barrier()
        return [stats([a.elapsed_time(b) for a, b in e]) for e in evs]

    def max_over_ranks(self, v):
        if self.world == 1:
            return v
        t = self.torch.tensor([v], dtype=self.torch.float64, device=self.dev)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())


def dense_comparators(h, api, torch, cfg, weights, layer, x, y, steps, step):
    """Same-shape dense FFN on the same tensors, same protocol: (1) torch eager F.linear -> act -> F.linear (cuBLASLt
    GEMMs, a separate activation kernel); (2) this library's own tensor-core GEMMs with every expert kept
    (bias + activation fused in the up projection's epilogue, no router, no selection); (3) the library's layer call
    at tau = 0 (router included, every expert kept).  The three and `step` (the measured configuration itself) are
    timed in one interleaved loop, and the speed-ups are ratios of medians from that loop."""
    import numpy as np
    import oracle
    dev = h.dev
    tdt = api.torch_dtype(cfg.dtype)
    F = torch.nn.functional
    w1 = torch.from_numpy(weights["w1"]).to(dev, tdt)
    w2 = torch.from_numpy(weights["w2"]).to(dev, tdt)
    b1 = None if weights["b1"] is None else torch.from_numpy(weights["b1"]).to(dev, tdt)
    b2 = None if weights["b2"] is None else torch.from_numpy(weights["b2"]).to(dev, tdt)
    wg = None if weights["w_gate"] is None else torch.from_numpy(weights["w_gate"]).to(dev, tdt)
    actf = {"relu": F.relu, "gelu_erf": F.gelu, "gelu_tanh": lambda z: F.gelu(z, approximate="tanh"), "silu": F.silu}[cfg.act]

    def dense():
        up = F.linear(x, w1, b1)
        hh = actf(F.linear(x, wg)) * up if wg is not None else actf(up)
        return F.linear(hh, w2, b2)

    T = x.shape[0]
    ones = np.ones((T, cfg.E), dtype=np.uint8)
    r_all = api.routing_from_mask(torch.from_numpy(oracle.pack_mask(ones).view(np.int32)).to(dev), cfg.E)
    path, group, rho_max = layer.get_expert_path()
    if cfg.dtype == "bf16":
        layer.set_expert_path("dense")
    r0 = layer.new_routing(T)
    y2 = torch.empty_like(y)
    # the graphs of the two library comparators are captured with the dense path forced, the step's own with its setting
    run_all = h.runner(lambda: layer.moe_ffn_fwd(x, r_all, y=y2))
    run_tau0 = h.runner(lambda: layer.layer_fwd(x, 0.0, y=y2, routing=r0))
    if cfg.dtype == "bf16":
        layer.set_expert_path(path, group, rho_max)
    run_step = h.runner(step)
    run_dense = h.runner(dense)
    no_graph, h.no_graph = h.no_graph, True                # the runners above are final: do not capture them again
    try:
        st = h.time_interleaved([run_step, run_dense, run_all, run_tau0], steps)
    finally:
        h.no_graph = no_graph
    out = {"step_interleaved_ms": st[0]["median"], "torch_eager_ms": st[1]["median"], "library_all_experts_ms": st[2]["median"],
           "library_layer_tau0_ms": st[3]["median"], "speedup": st[1]["median"] / st[0]["median"],
           "speedup_vs_library_dense": st[2]["median"] / st[0]["median"],
           "speedup_is": "torch eager dense FFN (cuBLASLt GEMMs + activation kernel) median / step median, one interleaved loop"}
    return out


def k_histogram(torch, routing, T, E):
    k = routing.k[:T].float()
    used = int((routing.counts > 0).sum().item()) if routing.lists else None
    return {"min": int(k.min().item()), "median": float(k.median().item()),
            "p99": float(torch.quantile(k, 0.99).item()), "max": int(k.max().item()), "experts_used": used}


def measure_config(h, api, torch, wl, name, tokens, tau, bern, steps, peaks, path="auto", group=0, full=False, rank=0, fp8=False):
    """One configuration: layer time, kept fraction, k histogram, dense comparators, roofline fraction of the expert step."""
    import numpy as np
    import oracle
    cfg = wl.CONFIGS[name]
    if tokens:
        cfg = wl.with_tokens(cfg, tokens)
    T = cfg.T
    dev = h.dev
    weights = wl.make_weights(cfg)
    x_np = wl.make_tokens(cfg, stream=rank)
    layer = api.Layer.from_config(cfg, weights, device=dev, fp8_experts=fp8)
    if cfg.dtype == "bf16" and (path != "auto" or group):
        layer.set_expert_path(path, group)
    x = api.to_device(x_np, cfg.dtype, dev)
    y = torch.empty_like(x)
    routing = layer.new_routing(T)
    layer.workspace(T)
    if bern is not None:
        G = wl.make_bernoulli_mask(cfg, bern, stream=rank)
        routing = api.routing_from_mask(torch.from_numpy(oracle.pack_mask(G).view(np.int32)).to(dev), cfg.E)

        def step():
            layer.moe_ffn_fwd(x, routing, y=y)
    else:
        def step():
            layer.layer_fwd(x, tau, y=y, routing=routing)
    step()
    l0 = api.launch_count()
    step()
    launches = api.launch_count() - l0
    res = {"cfg": cfg, "layer": layer, "weights": weights, "x": x, "x_np": x_np, "y": y, "routing": routing, "step": step,
           "launches": launches}
    if full:
        return res
    t = h.time(step, steps)
    torch.cuda.synchronize()
    assert routing.status == 0
    n_sel = routing.n_sel
    rho = n_sel / (T * cfg.E)
    dense = dense_comparators(h, api, torch, cfg, weights, layer, x, y, max(10, steps // 2), step)
    t_ffn = h.time(lambda: layer.moe_ffn_fwd(x, routing, y=y), max(10, steps // 2))["median"]
    f_experts = 2.0 * cfg.n_mat * cfg.d * cfg.s * n_sel
    elem = 2 if cfg.dtype == "bf16" else 4
    n_used = int((routing.counts > 0).sum().item())
    if T <= 64 or cfg.dtype == "f32":
        welem = 1 if fp8 else elem                           # 8-bit expert weights: one byte per weight
        touched = n_used * (cfg.n_mat * cfg.s * cfg.d * welem + cfg.s * elem) + 2 * T * cfg.d * elem + cfg.d * elem
        roof = {"bound": "hbm", "frac": touched / (t_ffn * 1e-3) / 1e9 / peaks["hbm_gbs"], "of": "touched expert bytes / expert-step time / HBM peak"}
    else:
        roof = {"bound": "tensor", "frac": f_experts / (t_ffn * 1e-3) / 1e12 / peaks["bf16_tflops"],
                "of": "algorithmic expert FLOP / expert-step time / bf16 peak"}
    out = {"workload": cfg.name, "tokens": T, "tau": tau, "bernoulli_p": bern, "expert_weights": "e4m3 + 2^k per expert" if fp8 else cfg.dtype, "rho": rho, "pruned_flop_fraction": 1 - rho,
           "k": k_histogram(torch, routing, T, cfg.E),
           "step": "d2d_moe_ffn_fwd on the override mask" if bern is not None else "d2d_layer_fwd",
           "ms_median": t["median"], "ms_min": t["min"], "tokens_per_s": T / (t["median"] * 1e-3),
           "expert_step_ms": t_ffn, "launches_per_step": launches, "expert_path": (layer.expert_path_for(T, n_sel) if launches > 2 else "decode kernels") if cfg.dtype == "bf16" else "fp32",
           "dense": dense, "speedup_vs_torch_dense": dense["speedup"],
           "speedup_vs_library_dense": dense["speedup_vs_library_dense"], "roofline": roof}
    layer.close()
    return out


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    import oracle
    from paper_2310_04361_b200 import api, workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the dynamic-k MoE layer has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    h = Harness(torch, dev, dist, world, args.no_graph)
    peaks = measured_peaks()

    m = measure_config(h, api, torch, wl, args.workload, args.tokens, args.tau, args.bernoulli, args.steps, peaks,
                       path=args.path, group=args.experts_per_group, full=True, rank=rank, fp8=args.fp8_experts)
    cfg, layer, weights, x, x_np, y, routing, step = (m[k] for k in ("cfg", "layer", "weights", "x", "x_np", "y", "routing", "step"))
    T = cfg.T
    launches_per_step = m["launches"]
    run_step = h.runner(step)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    times = h.timed_loop(run_step, args.steps, args.warmup)
    clocks = sampler.stop()
    total_ms = h.max_over_ranks(sum(times))
    value = world * T * args.steps / (total_ms * 1e-3)
    torch.cuda.synchronize()
    assert routing.status == 0
    n_sel = routing.n_sel
    rho = n_sel / (T * cfg.E)
    st_layer = stats(times)

    # ---- end to end through the host-buffer entry point (pinned host x -> device -> layer -> host y)
    e2e = None
    if args.bernoulli is None:
        xh = x.cpu().pin_memory()
        yh = torch.empty_like(xh).pin_memory()
        hws = layer.host_workspace(T)

        def e2e_step():
            layer.layer_fwd_host(xh, args.tau, yh, hws)

        for _ in range(max(3, args.warmup)):
            e2e_step()
        h.barrier()
        e2e_times = []
        for _ in range(args.steps):
            h.flush.zero_()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            e2e_step()                                 # synchronises the stream itself
            e2e_times.append(time.perf_counter() - t0)
        e2e_s = h.max_over_ranks(sum(e2e_times))
        row_bytes = T * cfg.d * (2 if cfg.dtype == "bf16" else 4)
        e2e = {"value": world * T * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": row_bytes,
               "d2h_bytes_per_step": row_bytes, "ms_median": 1e3 * sorted(e2e_times)[len(e2e_times) // 2],
               "note": "wall clock around each d2d_layer_fwd_host call (pinned host x and y; H2D copy, layer, D2H copy and "
                       "the stream synchronisation inside); the L2 flush before each call is outside the clock"}
        del hws

    line = None
    h.all_ranks = False                                    # what follows is measured by rank 0 alone
    if rank == 0:
        sub = max(10, args.steps // 2)
        # ---- per-stage breakdown (same protocol)
        stages = {"layer_fwd": st_layer["median"]}
        if args.bernoulli is None:
            R = torch.empty((T, cfg.E), dtype=torch.float32, device=dev)
            stages["router_fwd"] = h.time(lambda: layer.router_fwd(x, R=R), sub)["median"]
            r_tmp = layer.new_routing(T)
            stages["select_dynk"] = h.time(lambda: api.select_dynk(R, args.tau, routing=r_tmp), sub)["median"]
            del R, r_tmp
        t_ffn = h.time(lambda: layer.moe_ffn_fwd(x, routing, y=y), sub)["median"]
        stages["moe_ffn_fwd"] = t_ffn
        f_experts = 2.0 * cfg.n_mat * cfg.d * cfg.s * n_sel
        elem = 2 if cfg.dtype == "bf16" else 4
        n_used = int((routing.counts > 0).sum().item())
        if T <= 64 or cfg.dtype == "f32":
            # decode regime: the expert kernel is bound by HBM traffic on the touched expert slices
            welem = 1 if args.fp8_experts else elem           # 8-bit expert weights: one byte per weight
            touched = n_used * (cfg.n_mat * cfg.s * cfg.d * welem + cfg.s * elem) + 2 * T * cfg.d * elem + cfg.d * elem
            achieved = touched / (t_ffn * 1e-3) / 1e9
            roofline = {"bound": "hbm", "kernel": "moe_ffn_fwd (small_ffn_kernel)" if launches_per_step <= 2 else "moe_ffn_fwd", "achieved": achieved,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                        "peak_source": f"{peaks['source']} HBM copy", "algorithmic_bytes_per_launch": touched,
                        "experts_touched": n_used, "kernel_ms": t_ffn}
        else:
            # dominant kernel = the expert up projection; which of its two forms the step ran is the rule the kernels
            # themselves apply (n_sel against the layer's crossover); each is also timed on its own
            path, group, rho_max = layer.get_expert_path()
            taken = layer.expert_path_for(T, n_sel)            # the rule the kernels evaluate on the device
            gathered = taken in ("gather", "fused")
            H = torch.empty((T, cfg.d_ff), dtype=torch.bfloat16, device=dev)
            t_up_dense = h.time(lambda: layer.expert_up_fwd(x, routing, H=H), sub)["median"]
            t_up_gather = h.time(lambda: layer.expert_up_gather_fwd(x, routing, H=H), sub)["median"] if group > 0 else None
            layer.expert_up_fwd(x, routing, H=H)
            t_down = h.time(lambda: layer.expert_down_fwd(H, y=y), sub)["median"]
            t_down_masked = h.time(lambda: layer.expert_down_masked_fwd(H, routing, y=y), sub)["median"] if group > 0 else None
            t_up = t_up_gather if gathered else t_up_dense
            f_up = 2.0 * (cfg.n_mat - 1) * cfg.d * cfg.s * n_sel
            f_up_exec = 2.0 * (cfg.n_mat - 1) * T * cfg.d * cfg.d_ff
            if gathered:
                gmask = oracle.unpack_mask(routing.mask_u32(), cfg.E).reshape(T, cfg.E // group, group).max(-1)
                f_up_exec = 2.0 * (cfg.n_mat - 1) * cfg.d * cfg.s * group * float(gmask.sum())
            achieved = f_up / (t_up * 1e-3) / 1e12
            kname = "gather_up" if gathered else "dense_up"
            roofline = {"bound": "tensor",
                        "kernel": ("moe_gather_up_kernel (d2d_expert_up_gather_fwd)" if gathered else "gemm_tc_kernel<UP_MASKED> (d2d_expert_up_fwd)"),
                        "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                        "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, T, kname)),
                        "peak_source": f"{peaks['source']} burst bf16 GEMM", "algorithmic_flops_per_launch": f_up,
                        "executed_flops_per_launch": f_up_exec,
                        "executed_frac": f_up_exec / (t_up * 1e-3) / 1e12 / peaks["bf16_tflops"],
                        "kernel_ms": t_up, "up_dense_ms": t_up_dense, "up_gather_ms": t_up_gather, "down_dense_ms": t_down,
                        "down_masked_ms": t_down_masked, "expert_path": path, "path_taken": taken, "experts_per_group": group,
                        "expert_step_frac": f_experts / (t_ffn * 1e-3) / 1e12 / peaks["bf16_tflops"]}
            fgroup, frho = layer.get_fused()
            if taken == "fused":
                group = fgroup
                # one kernel does the whole expert step: its FLOPs are those of both projections over the kept pairs
                gmask = oracle.unpack_mask(routing.mask_u32(), cfg.E).reshape(T, cfg.E // group, group).max(-1)
                f_exec = 2.0 * cfg.n_mat * cfg.d * cfg.s * group * float(gmask.sum())
                roofline.update({"kernel": "moe_gather_ffn_kernel (d2d_moe_ffn_fwd, fused path; includes the accumulator's fill and conversion)",
                                 "achieved": f_experts / (t_ffn * 1e-3) / 1e12, "frac": f_experts / (t_ffn * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                 "algorithmic_flops_per_launch": f_experts, "executed_flops_per_launch": f_exec,
                                 "executed_frac": f_exec / (t_ffn * 1e-3) / 1e12 / peaks["bf16_tflops"], "kernel_ms": t_ffn,
                                 "merge_bytes_per_launch": 4.0 * cfg.d * float(gmask.sum()), "traffic": None})
            del H

        dense = dense_comparators(h, api, torch, cfg, weights, layer, x, y, sub, step)
        t_layer = st_layer["median"]

        sweep = None
        if args.sweep and args.bernoulli is None:
            sweep = []
            for tau in cfg.taus:
                ts = h.time(lambda tau=tau: layer.layer_fwd(x, tau, y=y, routing=routing), sub)
                torch.cuda.synchronize()
                sweep.append({"tau": tau, "rho": routing.n_sel / (T * cfg.E), "ms_median": ts["median"], "ms_min": ts["min"],
                              "speedup_vs_torch_dense": dense["torch_eager_ms"] / ts["median"],
                              "speedup_vs_library_dense": dense["library_all_experts_ms"] / ts["median"]})
            layer.layer_fwd(x, args.tau, y=y, routing=routing)
            torch.cuda.synchronize()

        group_res = None
        if args.group > 1:
            from dataclasses import replace
            tdt = api.torch_dtype(cfg.dtype)
            F = torch.nn.functional
            actf = {"relu": F.relu, "gelu_erf": F.gelu, "gelu_tanh": lambda z: F.gelu(z, approximate="tanh"), "silu": F.silu}[cfg.act]
            n = args.group
            gws = [weights] + [wl.make_weights(replace(cfg, seed=cfg.seed + 17 * l)) for l in range(1, n)]
            glayers = [layer] + [api.Layer.from_config(cfg, w, device=dev) for w in gws[1:]]
            grp = api.LayerGroup(glayers)
            gy = torch.empty((n, T, cfg.d), dtype=tdt, device=dev)
            grs = [L.new_routing(T) for L in glayers]
            grp.workspace(T)
            for L in glayers:
                L.workspace(T)

            def group_step():
                grp.group_fwd(x, args.tau, y=gy, routings=grs)

            def separate_step():
                for l, L in enumerate(glayers):
                    L.layer_fwd(x, args.tau, y=gy[l], routing=grs[l])

            gdense_w = [(torch.from_numpy(w["w1"]).to(dev, tdt), None if w["b1"] is None else torch.from_numpy(w["b1"]).to(dev, tdt),
                         torch.from_numpy(w["w2"]).to(dev, tdt), None if w["b2"] is None else torch.from_numpy(w["b2"]).to(dev, tdt))
                        for w in gws]

            def dense_group():
                return [F.linear(actf(F.linear(x, a, b)), c, e) for a, b, c, e in gdense_w]

            group_step()
            l0 = api.launch_count()
            group_step()
            g_launches = api.launch_count() - l0
            separate_step()
            l0 = api.launch_count()
            separate_step()
            s_launches = api.launch_count() - l0
            t_group = h.time(group_step, sub)["median"]
            t_sep = h.time(separate_step, sub)["median"]
            t_gdense = None if cfg.gated else h.time(dense_group, sub)["median"]
            torch.cuda.synchronize()
            assert all(r.status == 0 for r in grs)
            group_res = {"n_layers": n, "group_fwd_ms": t_group, "separate_layer_fwd_ms": t_sep, "dense_ms": t_gdense,
                         "launches_group": g_launches, "launches_separate": s_launches,
                         "speedup_vs_separate": t_sep / t_group, "speedup_vs_dense": None if t_gdense is None else t_gdense / t_group,
                         "rho": [r.n_sel / (T * cfg.E) for r in grs], "tokens_per_s": T / (t_group * 1e-3)}
            grp.close()

        khist = k_histogram(torch, routing, T, cfg.E)
        cpu = None
        if not args.no_cpu_baseline and args.bernoulli is None:
            cpu = time_cpu_oracle(cfg, weights, x_np, args.tau)
        layer.close()
        del layer, x, y, routing, weights
        torch.cuda.empty_cache()

        per_config = None
        if not args.no_per_config:
            per_config = []
            for name, tokens, tau, bern, *rest in PER_CONFIG:
                try:
                    per_config.append(measure_config(h, api, torch, wl, name, tokens, tau, bern, 20, peaks, fp8=bool(rest and rest[0])))
                except Exception as e:      # a configuration that fails must not take the headline down with it
                    per_config.append({"workload": name, "tokens": tokens, "tau": tau, "bernoulli_p": bern, "error": repr(e)})
                torch.cuda.empty_cache()

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "ms_median": st_layer["median"], "ms_min": st_layer["min"],
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype + (" (expert weights e4m3 + 2^k per expert)" if args.fp8_experts else ""), "data": "synthetic",
            "config": config_dict(cfg, args.tau, args.bernoulli),
            "run": {"tokens_per_gpu": T, "rho": rho, "pruned_flop_fraction": 1 - rho, "k": khist,
                    "step": "d2d_moe_ffn_fwd on the override mask" if args.bernoulli is not None else "d2d_layer_fwd",
                    "l2": f"flushed between steps by writing a {L2_FLUSH_BYTES >> 20} MiB buffer (outside the events)",
                    "launch": "eager" if args.no_graph else "CUDA graph replay of the library's launch sequence",
                    "parallelism": f"token-sharded replicas x{world}, no collective"},
            "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "clocks": clocks,
            "stages_ms": stages,
            "dense_ffn": dense,
            "paper_context": "paper reports ~3x over a dense MLP on an A100 at 99% accuracy (Sec. 4.4); another machine, not the target",
        }
        if per_config is not None:
            line["per_config"] = per_config
        if sweep is not None:
            line["tau_sweep"] = sweep
        if group_res is not None:
            line["group"] = group_res
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    args = parse_args()
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
