#!/usr/bin/env python
"""Benchmark of the dynamic-k MoE layer (D2DMoE inference hot path) on B200.

One step = one pass of the whole hot path (router_fwd -> select_dynk -> moe_ffn_fwd, the
single C-ABI call d2d_layer_fwd) over one batch of synthetic tokens.  Default workload: the
BERT-base-shaped bf16 layer (d=768, d_ff=3072, 128 experts x 24 neurons, 32 x 128 tokens).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--tau 0.3] [--workload bert] [--sweep]
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

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu
# capture summarised under profiles/ (None until a capture of that kernel/workload exists).
NCU_TRAFFIC_BYTES = {
    ("bert", 4096): 11.20e6,        # up projection: profiles/bert_gemm_up_down_full.md
    ("gpt2_ffn", 1, 0.2): 9.868e6,  # decode expert kernel: profiles/gpt2_decode_T1_small_kernels_full.md
}


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=50)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--workload", default="bert")
    p.add_argument("--tokens", type=int, default=0, help="override the workload's token count")
    p.add_argument("--tau", type=float, default=0.3)
    p.add_argument("--sweep", action="store_true", help="also time the workload's whole tau grid")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-graph", action="store_true", help="launch eagerly instead of replaying a captured CUDA graph")
    p.add_argument("--group", type=int, default=0,
                   help="also time N layers of the workload's shape on the shared input as one d2d_group_fwd call "
                        "(the Q, K, V projections of an attention layer) against N separate d2d_layer_fwd calls")
    return p.parse_args()


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


def flops_algorithmic(cfg, T, n_sel):
    router = 2.0 * T * (cfg.d * cfg.d_h + cfg.d_h * cfg.E)
    experts = 2.0 * cfg.n_mat * cfg.d * cfg.s * n_sel
    return router, experts


# ------------------------------------------------------------------------------------------ CPU oracle arm

def oracle_step_fn(cfg, weights, x_sample, tau):
    import oracle
    act = oracle.ACT_BY_NAME[cfg.act]

    def step():
        return oracle.layer(x_sample, weights, act, tau)
    return step


def time_cpu_oracle(cfg, weights, x, tau, budget_s=12.0):
    """Times the oracle, as it stands, on a bounded token sample sized for roughly budget_s seconds."""
    import oracle
    probe = min(32, x.shape[0])
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
    return {"value": n * passes / dt, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"first {n} of {x.shape[0]} tokens of the {cfg.name} workload at tau={tau}, {passes} passes "
                      f"(router+select+metadata+experts each), {dt:.2f} s"}


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
    probe = min(16, cfg.T)
    t0 = time.perf_counter()
    oracle_step_fn(cfg, weights, x[:probe], args.tau)()
    per_tok = (time.perf_counter() - t0) / probe
    total_steps = args.steps + args.warmup
    n = int(max(1, min(cfg.T, 90.0 / total_steps / max(per_tok, 1e-9))))   # whole run within ~1.5 minutes
    step = oracle_step_fn(cfg, weights, x[:n], args.tau)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = n * args.steps / dt
    sample = f"each step = the first {n} of {cfg.T} tokens of the {cfg.name} workload at tau={args.tau}"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "tokens_per_step": n, "d": cfg.d, "d_ff": cfg.d_ff, "experts": cfg.E,
                   "expert_size": cfg.s, "d_h": cfg.d_h, "act": cfg.act, "tau": args.tau},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


# ------------------------------------------------------------------------------------------ GPU arm

def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
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

    cfg = wl.CONFIGS[args.workload]
    if args.tokens:
        cfg = wl.with_tokens(cfg, args.tokens)
    T = cfg.T
    weights = wl.make_weights(cfg)                      # every rank holds the whole layer
    x_np = wl.make_tokens(cfg, stream=rank)             # ... and its own batch of tokens
    layer = api.Layer.from_config(cfg, weights, device=dev)
    x = api.to_device(x_np, cfg.dtype, dev)
    y = torch.empty_like(x)
    routing = layer.new_routing(T)
    layer.workspace(T)
    flush = torch.empty((L2_FLUSH_BYTES,), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_loop(fn, steps, warmup):
        """Per-step CUDA events on the launching stream; the L2 flush between steps is outside the events."""
        for _ in range(warmup):
            flush.zero_()
            fn()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        barrier()
        for a, b in evs:
            flush.zero_()
            a.record(stream)
            fn()
            b.record(stream)
        barrier()
        return [a.elapsed_time(b) for a, b in evs]       # ms

    def runner(fn):
        """The step as it is launched in the timed region: a CUDA-graph replay of the library's launch
        sequence (the layer is launch-latency bound for small batches), or the eager call with --no-graph."""
        if args.no_graph:
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

    def max_over_ranks(v):
        if world == 1:
            return v
        t = torch.tensor([v], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def step():
        layer.layer_fwd(x, args.tau, y=y, routing=routing)

    step()                                   # one eager call: counts the kernels a step launches
    launches0 = api.launch_count()
    step()
    launches_per_step = api.launch_count() - launches0
    run_step = runner(step)
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    times = timed_loop(run_step, args.steps, args.warmup)
    clocks = sampler.stop()
    total_ms = max_over_ranks(sum(times))
    value = world * T * args.steps / (total_ms * 1e-3)
    torch.cuda.synchronize()
    n_sel = routing.n_sel
    assert routing.status == 0

    # ---- end to end through the host-buffer entry point (pinned host x -> device -> layer -> host y)
    xh = x.cpu().pin_memory()
    yh = torch.empty_like(xh).pin_memory()
    hws = layer.host_workspace(T)

    def e2e_step():
        layer.layer_fwd_host(xh, args.tau, yh, hws)

    for _ in range(max(3, args.warmup)):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        flush.zero_()
        e2e_step()
    torch.cuda.synchronize()
    e2e_s = max_over_ranks(time.perf_counter() - t0)
    row_bytes = T * cfg.d * (2 if cfg.dtype == "bf16" else 4)
    e2e = {"value": world * T * args.steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": row_bytes,
           "d2h_bytes_per_step": row_bytes, "note": "wall clock over K calls of d2d_layer_fwd_host incl. an L2 flush per step"}

    line = None
    if rank == 0:
        # ---- per-stage breakdown (same flush protocol), used for the roofline of the dominant kernel
        R = torch.empty((T, cfg.E), dtype=torch.float32, device=dev)
        t_router = statistics.mean(timed_loop(runner(lambda: layer.router_fwd(x, R=R)), args.steps, 3))
        t_select = statistics.mean(timed_loop(runner(lambda: api.select_dynk(R, args.tau, routing=routing)), args.steps, 3))
        t_ffn = statistics.mean(timed_loop(runner(lambda: layer.moe_ffn_fwd(x, routing, y=y)), args.steps, 3))
        peaks = measured_peaks()
        f_router, f_experts = flops_algorithmic(cfg, T, n_sel)
        elem = 2 if cfg.dtype == "bf16" else 4
        n_used = int((routing.counts > 0).sum().item())
        if T <= 64 or cfg.dtype == "f32":
            # decode regime: the expert kernel is bound by HBM traffic on the touched expert slices
            touched = n_used * (cfg.n_mat * cfg.s * cfg.d + cfg.s) * elem + 2 * T * cfg.d * elem + cfg.d * elem
            achieved = touched / (t_ffn * 1e-3) / 1e9
            roofline = {"bound": "hbm", "kernel": "moe_ffn_fwd (small_ffn_kernel)" if T <= 4 else "moe_ffn_fwd", "achieved": achieved,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                        "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, T, args.tau)),
                        "peak_source": f"{peaks['source']} HBM copy", "algorithmic_bytes_per_launch": touched,
                        "experts_touched": n_used, "kernel_ms": t_ffn}
        else:
            # dominant kernel = the expert up projection (one launch of gemm_tc_kernel with the masked
            # activation epilogue); its algorithmic work is the up half of the kept pairs' FLOP
            H = torch.empty((T, cfg.d_ff), dtype=torch.bfloat16, device=dev)
            t_up = statistics.mean(timed_loop(runner(lambda: layer.expert_up_fwd(x, routing, H=H)), args.steps, 3))
            t_down = statistics.mean(timed_loop(runner(lambda: layer.expert_down_fwd(H, y=y)), args.steps, 3))
            f_up = 2.0 * (cfg.n_mat - 1) * cfg.d * cfg.s * n_sel
            f_up_exec = 2.0 * (cfg.n_mat - 1) * T * cfg.d * cfg.d_ff
            achieved = f_up / (t_up * 1e-3) / 1e12
            roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel<UP_MASKED> (d2d_expert_up_fwd)", "achieved": achieved,
                        "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                        "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, T)),
                        "peak_source": f"{peaks['source']} burst bf16 GEMM", "algorithmic_flops_per_launch": f_up,
                        "executed_flops_per_launch": f_up_exec,
                        "executed_frac": f_up_exec / (t_up * 1e-3) / 1e12 / peaks["bf16_tflops"],
                        "kernel_ms": t_up, "down_kernel_ms": t_down,
                        "expert_step_frac": f_experts / (t_ffn * 1e-3) / 1e12 / peaks["bf16_tflops"]}

        # ---- dense FFN comparator: torch (cuBLASLt) linear -> act -> linear on the same tensors
        tdt = api.torch_dtype(cfg.dtype)
        w1 = torch.from_numpy(weights["w1"]).to(dev, tdt)
        w2 = torch.from_numpy(weights["w2"]).to(dev, tdt)
        b1 = None if weights["b1"] is None else torch.from_numpy(weights["b1"]).to(dev, tdt)
        b2 = None if weights["b2"] is None else torch.from_numpy(weights["b2"]).to(dev, tdt)
        wg = None if weights["w_gate"] is None else torch.from_numpy(weights["w_gate"]).to(dev, tdt)
        F = torch.nn.functional
        actf = {"relu": F.relu, "gelu_erf": F.gelu, "gelu_tanh": lambda z: F.gelu(z, approximate="tanh"), "silu": F.silu}[cfg.act]

        def dense():
            up = F.linear(x, w1, b1)
            h = actf(F.linear(x, wg)) * up if wg is not None else actf(up)
            return F.linear(h, w2, b2)

        t_dense = statistics.mean(timed_loop(runner(dense), args.steps, 3))
        t_layer = sum(times) / len(times)

        sweep = None
        if args.sweep:
            sweep = []
            for tau in cfg.taus:
                ts = timed_loop(runner(lambda tau=tau: layer.layer_fwd(x, tau, y=y, routing=routing)), max(10, args.steps // 2), 3)
                torch.cuda.synchronize()
                sweep.append({"tau": tau, "rho": routing.n_sel / (T * cfg.E), "ms": statistics.mean(ts),
                              "speedup_vs_dense": t_dense / statistics.mean(ts)})

        group = None
        if args.group > 1:
            from dataclasses import replace
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
            t_group = statistics.mean(timed_loop(runner(group_step), args.steps, 3))
            t_sep = statistics.mean(timed_loop(runner(separate_step), args.steps, 3))
            t_gdense = None if cfg.gated else statistics.mean(timed_loop(runner(dense_group), args.steps, 3))
            torch.cuda.synchronize()
            assert all(r.status == 0 for r in grs)
            group = {"n_layers": n, "group_fwd_ms": t_group, "separate_layer_fwd_ms": t_sep, "dense_ms": t_gdense,
                     "launches_group": g_launches, "launches_separate": s_launches,
                     "speedup_vs_separate": t_sep / t_group, "speedup_vs_dense": None if t_gdense is None else t_gdense / t_group,
                     "rho": [r.n_sel / (T * cfg.E) for r in grs],
                     "tokens_per_s": T / (t_group * 1e-3)}
            grp.close()

        cpu = None
        if not args.no_cpu_baseline:
            cpu = time_cpu_oracle(cfg, weights, x_np, args.tau)

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "tokens_per_gpu": T, "d": cfg.d, "d_ff": cfg.d_ff, "experts": cfg.E,
                       "expert_size": cfg.s, "d_h": cfg.d_h, "act": cfg.act, "gated": cfg.gated, "tau": args.tau,
                       "rho": n_sel / (T * cfg.E), "pruned_flop_fraction": 1 - n_sel / (T * cfg.E),
                       "l2": f"flushed between steps by writing a {L2_FLUSH_BYTES >> 20} MiB buffer (outside the events)",
                       "launch": "eager" if args.no_graph else "CUDA graph replay of the library's launch sequence",
                       "parallelism": f"token-sharded replicas x{world}, no collective"},
            "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "clocks": clocks,
            "stages_ms": {"router_fwd": t_router, "select_dynk": t_select, "moe_ffn_fwd": t_ffn, "layer_fwd": t_layer},
            "dense_ffn": {"ms": t_dense, "impl": "torch F.linear/act/F.linear (cuBLASLt)", "speedup_of_layer": t_dense / t_layer,
                          "speedup_of_moe_ffn_only": t_dense / t_ffn},
            "paper_context": "paper reports ~3x over a dense MLP on an A100 at 99% accuracy (Sec. 4.4); another machine, not the target",
        }
        if sweep is not None:
            line["tau_sweep"] = sweep
        if group is not None:
            line["group"] = group
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
