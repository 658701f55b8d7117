#!/usr/bin/env python
"""Benchmark of the complete-expert MoE layer forward on B200 (one process per GPU).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the whole hot path (grouping, gate/up GEMM + SwiGLU, down GEMM, combine; plus
resolution and miss copies when slots < experts) over one batch of synthetic tokens of one
OLMoE-shaped sparse layer.  Default workload: decode, 1 token per step, 64 slots (fully resident),
fresh seeded hidden state per step, rotating over 16 independent layer banks (3.3 GB of packed
experts) so that every step's weights come from HBM, not from the 126 MB L2.

Prints ONE JSON line: MoE-layer tokens/s (inputs resident in HBM, CUDA-graph replay, CUDA events),
the end-to-end number through host buffers, the roofline of the dominant kernel (gate/up GEMM;
packed weight + scale bytes it must read / its CUDA-event time / measured HBM copy rate) and of the
whole step, the CPU oracle timed on the host cores on a bounded sample, SM clocks sampled during the
timed region and the number of kernels launched.  The timed region is long whatever --steps is: the
graph of K steps is replayed until a repetition lasts at least 60 ms, five repetitions are taken and
the median is reported (with the spread), so that the clocks are up and the sampler sees the region.
The default (decode) run then adds two short legs to the same line: `config.prefill` (config 4,
tensor-core roofline) and `config.offload` (config 3, host-link roofline), plus the pack throughput.
`--impl reference` times the CPU oracle alone.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2608_15383_b200 import synth

WORKLOADS = {
    # name: (tokens per step, slots, layers rotated over, Zipf alpha, description)
    "decode": (1, 64, 16, 0.0, "config2: OLMoE-shaped decode, T=1, 64 slots resident, top-8 of 64, int4 g128"),
    "decode16": (16, 64, 16, 1.0, "OLMoE-shaped batched decode, T=16, 64 slots resident, Zipf(1.1) routing"),
    "offload": (16, 16, 1, "cycle", "config3: T=16, 16 slots over a 64-expert pinned host bank, Zipf(1.1) routing bias "
                "x alpha, alpha cycling over {2, 1, 0.5, 0} in four blocks of steps (1-4 waves per step)"),
    "prefill": (2048, 64, 1, 0.0, "config4: OLMoE-shaped prefill, T=2048, 64 slots resident, uniform routing"),
}
# DRAM bytes (read + write) per launch of the dominant kernel, from one ncu capture each (dram__bytes_read.sum +
# dram__bytes_write.sum, two layer banks = 415 MB resident; per-launch traffic does not depend on the number of banks):
# (bytes, kernel captured, date of the capture)
NCU_TRAFFIC = {"decode": (17.33e6, "pair_gateup_wide_kernel<4>, T=1", "2026-11-25"),
               "decode16": (62.83e6 + 0.87e6, "stream_gemm_kernel<1,true,1>, T=16", "2026-11-25"),
               "prefill": (215.63e6 + 11.33e6, "prefill_gemm_kernel<true,256,4>, T=2048", "2026-11-25")}
METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """SM clock and throttle reasons of this rank's GPU while the timed region runs.  Read-only NVML queries from a
    sampling thread every ~5 ms (every timed region lasts hundreds of ms); falls back to
    `nvidia-smi -lms 100` when the NVML binding is missing."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.p, self.f, self.thread = None, None, None
        self.sm, self.mx, self.reasons = [], [], set()
        try:
            import pynvml
            import threading
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByIndex(int(index))
            bits = {"hw_slowdown": pynvml.nvmlClocksThrottleReasonHwSlowdown,
                    "hw_thermal_slowdown": pynvml.nvmlClocksThrottleReasonHwThermalSlowdown,
                    "sw_thermal_slowdown": pynvml.nvmlClocksThrottleReasonSwThermalSlowdown,
                    "sw_power_cap": pynvml.nvmlClocksThrottleReasonSwPowerCap}
            mx = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self.stop_flag = threading.Event()

            def loop():
                while not self.stop_flag.is_set():
                    try:
                        self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        self.mx.append(mx)
                        r = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                        for n, b in bits.items():
                            if r & b:
                                self.reasons.add(n)
                    except Exception:
                        pass
                    time.sleep(0.005)
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.thread = None
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def mark(self):
        """Drop what was sampled so far: called right before the timed region starts (NVML sampler only)."""
        if self.thread is not None:
            del self.sm[:], self.mx[:]
            self.reasons.clear()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            if self.sm:
                out.update(sm_mhz=float(np.median(self.sm)), sm_max_mhz=float(max(self.mx)), reasons=sorted(self.reasons),
                           samples=len(self.sm), source="nvml, 5 ms period")
            return out
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm),
                       source="nvidia-smi, 100 ms period")
        return out


def max_over_ranks(x, world, device="cpu"):
    """Slowest rank's value (device time of the timed region): the job is as fast as its slowest replica."""
    if world <= 1:
        return float(x)
    import torch.distributed as dist
    t = torch.tensor([float(x)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(world, steps, tokens_per_step, ms_max):
    """Replicas only (no collective on the data path): every rank runs the same workload on its own GPU."""
    return world * steps * tokens_per_step / (ms_max * 1e-3)


def make_inputs(shape, T, n_sets, alpha, seed0, device):
    """n_sets independent (hidden, ids, weights) batches, generated on the device and routed by Eq. 1: by the library's
    router kernel (exmoe_route) on a GPU, by the oracle's router on the CPU (the reference arm runs without a GPU).
    alpha = "cycle": the sets fall into four consecutive blocks with alpha = 2, 1, 0.5, 0 (same rank permutation)."""
    if str(device) == "cpu":
        from oracle import router as orouter

        def route(h, wr, k, bias):
            ids, p, _ = orouter.route(h.float().numpy(), wr.float().numpy(), k, None if bias is None else bias.numpy())
            return torch.from_numpy(ids), torch.from_numpy(p.astype(np.float32))
    else:
        from paper_2608_15383_b200 import binding

        def route(h, wr, k, bias):
            return binding.exmoe_route(shape, h, wr, None if bias is None else bias.float().contiguous())
    wr = synth.router_weights(shape, seed0 + 1, device=device)
    cycle = (2.0, 1.0, 0.5, 0.0)
    base = synth.zipf_bias(shape.num_experts, 1.0, seed0 + 2).to(device)
    hs, ids, ws = [], [], []
    for i in range(n_sets):
        al = cycle[min(3, i * 4 // max(n_sets, 1))] if alpha == "cycle" else float(alpha)
        bias = base * al if al else None
        h = synth.hidden_states(shape, T, seed0 + 10 + i, device=device)
        a, b = route(h, wr, shape.top_k, bias)
        hs.append(h)
        ids.append(a)
        ws.append(b)
    return hs, ids, ws


PACK_STATS = {}


def build_banks(shape, layers, seed0, device, keep_layer0=False):
    """Per layer: draw BF16 expert weights on the device, pack them with exmoe_pack into a pinned host bank.
    The last layer's packing (exmoe_pack alone, device buffers in and out, host clock around a synchronised loop) is timed."""
    from paper_2608_15383_b200 import binding
    banks, kept = [], None
    for l in range(layers):
        wg, wu, wd = synth.expert_weights(shape, seed0 + l, device=device)
        banks.append(binding.pack_bank(shape, wg, wu, wd, device=device))
        if l == layers - 1:
            buf = torch.empty(binding.exmoe_packed_bytes(shape), dtype=torch.uint8, device=device)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for e in range(shape.num_experts):
                binding.exmoe_pack(shape, wg[e], wu[e], wd[e], buf)
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            read = 3 * shape.d_ff * shape.d_model * 2
            PACK_STATS.update({"experts_per_s": shape.num_experts / dt, "bf16_gb_read_per_s": shape.num_experts * read / dt / 1e9,
                               "us_per_expert": 1e6 * dt / shape.num_experts,
                               "note": "exmoe_pack, one synchronous call per expert (the status covers the data)"})
        if l == 0 and keep_layer0:
            kept = (wg.cpu(), wu.cpu(), wd.cpu())
        del wg, wu, wd
    return banks, kept


def oracle_leg(shape, T, weights_cpu, hs, ids, ws, budget_s):
    """Time the CPU oracle as it stands on batches of the same workload until ~budget_s of work is done."""
    from oracle import moe as omoe, quant as oquant
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = 1
    wg, wu, wd = weights_cpu
    cache = {}

    def expert(e):
        if e not in cache:
            if len(cache) >= 24:
                cache.pop(next(iter(cache)))
            cache[e] = tuple(oquant.dequantize_g128(*oquant.quantize_g128(w[e].float().numpy())) for w in (wg, wu, wd))
        return cache[e]

    done_tokens, t0, steps = 0, time.perf_counter(), 0
    t_rows = min(T, 8)                                   # a bounded sample of each batch's tokens
    while steps < len(hs):
        h = hs[steps][:t_rows].float().cpu().numpy()
        i = ids[steps][:t_rows].cpu().numpy()
        w = ws[steps][:t_rows].cpu().numpy()
        omoe.moe_layer_forward(h, i, w, expert, shape.num_experts)
        done_tokens += t_rows
        steps += 1
        if time.perf_counter() - t0 > budget_s:
            break
    dt = time.perf_counter() - t0
    return {"value": done_tokens / dt, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": f"{steps} steps x {t_rows} tokens of layer 0 ({done_tokens} tokens, {dt:.1f} s), dequantising on the fly"}


def run_reference(args, rank, world):
    if rank != 0:
        return
    T, C, L, alpha, desc = WORKLOADS[args.workload]
    shape = synth.OLMOE
    wg, wu, wd = synth.expert_weights(shape, 2000, device="cpu")
    hs, ids, ws = make_inputs(shape, T, max(args.steps + args.warmup, 4), alpha, 2000, "cpu")
    per_step_budget = max(2.0, 120.0 / max(args.steps + args.warmup, 1))
    from oracle import moe as omoe, quant as oquant
    leg = None
    for _ in range(args.warmup):                         # one bounded-sample step each
        oracle_leg(shape, T, (wg, wu, wd), hs[:1], ids[:1], ws[:1], 0.0)
    t0 = time.perf_counter()
    tokens = 0
    for s in range(args.steps):
        leg = oracle_leg(shape, T, (wg, wu, wd), hs[s:s + 1], ids[s:s + 1], ws[s:s + 1], per_step_budget)
        tokens += min(T, 8)
    dt = time.perf_counter() - t0
    value = tokens / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(args.steps, 1), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": desc, "note": "CPU oracle on a bounded sample: first min(T,8) tokens of each step",
                       "steps_requested": args.steps_requested},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": leg["cores"] if leg else 1, "kind": "oracle",
                             "sample": f"{args.steps} steps x {min(T, 8)} tokens"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_stack_sweep(args, dev, binding):
    """Config 5: 16-layer stack (synthetic routers + identity-plus-noise residual), decode batch sweep x slot
    sweep, Zipf-skewed routing.  Reports tokens/s, expert H2D bytes per token and peak reserved GPU memory."""
    shape, L = synth.OLMOE, args.layers or 16
    banks, _ = build_banks(shape, L, 5000, dev)
    rows = []
    for C in (16, 32, 64):
        for T in (1, 4, 16, 64):
            torch.cuda.empty_cache()
            torch.cuda.reset_peak_memory_stats(dev)
            cache = binding.Cache(shape, banks, C, max_tokens=64, device=dev)
            device_fetch = args.miss_path == "device" and C < shape.num_experts
            if C < shape.num_experts:
                cache.set_miss_path(binding.MISS_DEVICE_FETCH if device_fetch else binding.MISS_HOST_COPIES)
            stack = synth.SyntheticStack(shape, L, seed=5100, alpha=(0.5 if args.alpha is None else args.alpha), device=dev)
            # every step decodes fresh tokens: a new seeded hidden state enters layer 0 (as an embedding would)
            pool = [synth.hidden_states(shape, T, 5200 + i, device=dev) for i in range(16)]
            fwd = lambda l, x, ids, w: cache.forward(l, x, ids, w)
            bias32 = [None if b is None else b.float().contiguous() for b in stack.bias]
            # the library's fused router (Eq. 1) on the current stream instead of the harness's torch router
            rt = lambda l, x: binding.exmoe_route(shape, x, stack.routers[l], bias32[l])
            # next-layer prefetch policy: layer l+1's router applied to layer l's input, on a side stream; layer l+1's
            # forward waits for that prefetch (an event), layer l's kernels run beside it
            # (only while the guessed set fits the layer's slots: a larger prefetch would evict its own first wave)
            use_pf = args.prefetch and device_fetch and T * shape.top_k <= C
            pf_side = torch.cuda.Stream(device=dev) if use_pf else None
            pf_done = {}

            def make_hooks(main_stream):
                if not use_pf:
                    return None, (lambda l, x, ids, w: cache.forward(l, x, ids, w, stream=main_stream))

                def look(l_next, x):
                    ready = torch.cuda.Event()
                    ready.record(main_stream)
                    pf_side.wait_event(ready)
                    x.record_stream(pf_side)                       # the side stream reads the layer input after this call returns
                    with torch.cuda.stream(pf_side):
                        guess, _ = binding.exmoe_route(shape, x, stack.routers[l_next], bias32[l_next], stream=pf_side)
                        cache.prefetch(l_next, guess, stream=pf_side)
                        ev = torch.cuda.Event()
                        ev.record(pf_side)
                    pf_done[l_next] = ev

                def fwd_pf(l, x, ids, w):
                    ev = pf_done.pop(l, None)
                    if ev is not None:
                        main_stream.wait_event(ev)
                    return cache.forward(l, x, ids, w, stream=main_stream)
                return look, fwd_pf
            warm, timed = (args.warmup or 16), (args.steps if args.steps < 1000 else 64)
            look0, fwd0 = make_hooks(torch.cuda.current_stream())
            if use_pf:
                fwd = fwd0
            for i in range(warm):
                h = stack.step(fwd, pool[i % 16], route_fn=rt, lookahead_fn=look0)
            torch.cuda.synchronize()
            graph = None
            if C == shape.num_experts or device_fetch:    # no host wait inside the layer call: the step is graph-capturable
                # residual noise of all layers in one tensor the graph reads; redrawn before every replay (two launches),
                # so that the replayed steps see the same random walk as host-driven ones
                noise_all = torch.empty((L, T, shape.d_model), device=dev, dtype=torch.float32)
                noise_all.normal_(generator=stack.gen).mul_(0.1)
                noise = list(noise_all.unbind(0))
                h_in = pool[0].clone()
                side = torch.cuda.Stream(device=dev)
                look_s, fwd_s = make_hooks(side)
                with torch.cuda.stream(side):
                    stack.step(fwd_s, h_in, noise=noise, route_fn=rt, lookahead_fn=look_s)
                side.synchronize()
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    h = stack.step(fwd_s, h_in, noise=noise, route_fn=rt, lookahead_fn=look_s)
                graph.replay()
                torch.cuda.synchronize()
            st0 = [cache.stats(l) for l in range(L)]
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(timed):
                if graph is not None:
                    h_in.copy_(pool[(warm + i) % 16])
                    noise_all.normal_(generator=stack.gen).mul_(0.1)
                    graph.replay()
                else:
                    h = stack.step(fwd, pool[(warm + i) % 16], route_fn=rt, lookahead_fn=look0)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / timed
            st1 = [cache.stats(l) for l in range(L)]
            d = lambda key: sum(b[key] - a[key] for a, b in zip(st0, st1))
            rows.append({"slots": C, "tokens": T, "tokens_per_s": T / (ms * 1e-3), "ms_per_step": ms,
                         "h2d_bytes_per_token": d("h2d_bytes") / (timed * T),
                         "hit_rate": (d("hits") / d("lookups")) if d("lookups") else None,
                         "waves_per_layer_call": (d("waves") / d("forwards")) if d("forwards") else 1.0,
                         "peak_reserved_gib": torch.cuda.max_memory_reserved(dev) / 2 ** 30,
                         "prefetch": bool(use_pf),
                         "miss_path": "device fetch" if device_fetch else ("host copies" if C < shape.num_experts else None),
                         "timing": "CUDA graph of the 16-layer step" if graph is not None else "host-driven"})
            assert cache.status() == 0 and bool(torch.isfinite(h.float()).all())
            cache.close()
            del cache
            print(json.dumps(rows[-1]), file=sys.stderr, flush=True)
    return rows


MIN_REGION_MS = 60.0      # a timed repetition replays the K-step graph until it lasts at least this long
REPS = 5                  # repetitions; the median is reported


def timed_repetitions(stream, run_once, ms_hint=None):
    """CUDA-event time of `run_once` (one graph replay of K steps, or K host-driven steps), repeated back to back until
    a repetition lasts MIN_REGION_MS, REPS repetitions.  Returns (list of ms per call of run_once, calls per repetition)."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        run_once()
        e1.record(stream)
    stream.synchronize()
    one = max(e0.elapsed_time(e1), 1e-3)
    m = int(min(max(1, np.ceil(MIN_REGION_MS / one)), 20000))
    out = []
    for _ in range(REPS):
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(m):
                run_once()
            e1.record(stream)
        stream.synchronize()
        out.append(e0.elapsed_time(e1) / m)
    return out, m


def run_leg(name, args, shape, banks, dev, rank, local_rank, world, peaks, K, W, seed0, full):
    """One workload through the device-timed path (and, if `full`, the per-kernel, end-to-end and copy-link parts).
    Returns a dict with value, ms_per_step, roofline, kernel_us, clocks, launches and descriptive fields."""
    import torch.distributed as dist
    from paper_2608_15383_b200 import binding
    T, C, L, alpha, desc = WORKLOADS[name]
    L = min(args.layers or L, len(banks))
    if full and args.tokens:
        T, desc = args.tokens, desc + " [tokens per step overridden: %d]" % args.tokens
    if full and args.slots:
        C, desc = args.slots, desc + " [slots overridden: %d]" % args.slots
    if full and args.alpha is not None:
        alpha, desc = args.alpha, desc + " [routing skew alpha overridden: %g]" % args.alpha
    cache = binding.Cache(shape, banks[:L], C, max_tokens=T, device=dev)
    if C < shape.num_experts:
        cache.set_miss_path(binding.MISS_DEVICE_FETCH if args.miss_path == "device" else binding.MISS_HOST_COPIES)
        desc += " [miss path: %s]" % ("device-initiated fetch kernel" if args.miss_path == "device" else "host-issued copies")
    n_sets = min(K + W, 1024) if T <= 64 else 4
    hs, ids, ws = make_inputs(shape, T, n_sets, alpha, seed0, dev)
    outs = [torch.empty_like(hs[0]) for _ in range(2)]
    stream = torch.cuda.Stream(device=dev)
    identity = (C == shape.num_experts)
    graphable = identity or args.miss_path == "device"       # no host wait inside the call: the steps replay from a graph

    def step(i, out):
        cache.forward(i % L, hs[i % n_sets], ids[i % n_sets], ws[i % n_sets], out=out, stream=stream)

    with torch.cuda.stream(stream):
        for i in range(3):
            step(i, outs[0])
    stream.synchronize()

    # ---- device-timed region: CUDA-graph replay of the K steps (no host sync inside), repeated (see timed_repetitions)
    if graphable:
        graph_w, graph_k = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_w, stream=stream):
            for i in range(W):
                step(i, outs[i & 1])
        launches0 = binding.exmoe_launch_count()
        with torch.cuda.graph(graph_k, stream=stream):
            for i in range(W, W + K):
                step(i, outs[i & 1])
        launches = binding.exmoe_launch_count() - launches0
        with torch.cuda.stream(stream):
            graph_w.replay()
            graph_k.replay()          # untimed first replay: uploads the instantiated graph to the device
        run_once = graph_k.replay
    else:
        with torch.cuda.stream(stream):
            for i in range(W):
                step(i, outs[i & 1])
        launches0 = binding.exmoe_launch_count()
        with torch.cuda.stream(stream):
            for i in range(W, W + K):
                step(i, outs[i & 1])
        launches = binding.exmoe_launch_count() - launches0

        def run_once():
            for i in range(W, W + K):
                step(i, outs[i & 1])
    stream.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local_rank)
    stats0 = cache.stats(0) if not identity else None
    sampler.mark()
    reps_ms, replays = timed_repetitions(stream, run_once)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    ms = max_over_ranks(float(np.median(reps_ms)), world, dev)              # ms per K steps, slowest rank's median
    value = whole_job_tokens_per_s(world, K, T, ms)
    ms_step = ms / K
    if clocks.get("sm_mhz"):
        clocks["us_per_step_x_sm_ghz"] = 1e3 * ms_step * clocks["sm_mhz"] / 1e3   # kcycles per step: compare across clock states

    res = {"name": name, "desc": desc, "T": T, "C": C, "L": L, "K": K, "W": W, "value": value, "ms_per_step": ms_step,
           "launches": int(launches), "clocks": clocks, "graphable": graphable,
           "repetitions": {"count": REPS, "replays_of_the_K_step_graph_each": replays,
                           "ms_per_step_min_median_max": [min(reps_ms) / K, float(np.median(reps_ms)) / K, max(reps_ms) / K],
                           "region_ms_each": float(np.median(reps_ms)) * replays}}

    # ---- per-kernel times (roofline of the dominant kernel): the same steps with ONLY one kernel kind
    # launched, timed with CUDA events on the launching stream (graph replay when graphable), same repetition rule
    n_prof = min(K, 200)
    kinds = {}
    for kind, kname in ((1, "gate_up"), (2, "down")):
        cache.profile_enable(False, only=kind)
        with torch.cuda.stream(stream):
            step(0, outs[0])
        stream.synchronize()
        if identity:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for i in range(W, W + n_prof):
                    step(i, outs[i & 1])
            with torch.cuda.stream(stream):
                g.replay()
            kms, _ = timed_repetitions(stream, g.replay)
        else:
            def only_once():
                for i in range(W, W + n_prof):
                    step(i, outs[i & 1])
            kms, _ = timed_repetitions(stream, only_once)
        kinds[kname] = {"us_per_launch": 1e3 * float(np.median(kms)) / n_prof, "launches_per_replay": n_prof}
    cache.profile_enable(False)
    bpe = cache.bytes_per_expert
    w13_bytes = bpe * 2 // 3
    active = float(np.mean([len(torch.unique(ids[i % n_sets])) for i in range(W, W + n_prof)]))      # the steps timed above
    active_all = float(np.mean([len(torch.unique(ids[i % n_sets])) for i in range(W, W + K, max(K // 200, 1))]))
    step_gbs = active_all * bpe / (ms_step * 1e-3) / 1e9
    flops_step = 2.0 * T * shape.top_k * 3 * shape.d_ff * shape.d_model
    step_tflops = flops_step / (ms_step * 1e-3) / 1e12
    traffic = NCU_TRAFFIC.get(name) if not (full and (args.tokens or args.slots)) else None
    if T * shape.top_k > 640:
        flops = 2.0 * T * shape.top_k * 2 * shape.d_ff * shape.d_model          # gate/up GEMM of one step
        achieved = flops / (kinds["gate_up"]["us_per_launch"] * 1e-6) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac": achieved / peaks["bf16_tflops"], "traffic": traffic[0] if traffic else None,
                "traffic_unit": "bytes per launch (ncu dram read + write)",
                "traffic_source": ("one ncu capture of %s on %s" % traffic[1:]) if traffic else None,
                "kernel": "gate_up (prefill_gemm_kernel<true>, tcgen05)", "flops_per_launch": flops,
                "peak_source": peaks["source"] + " cuBLAS bf16, burst",
                "whole_step": {"achieved": step_tflops, "flops_per_step": flops_step, "frac": step_tflops / peaks["bf16_tflops"],
                               "frac_of_sustained": step_tflops / peaks["bf16_tflops_sustained"]}}
    else:
        gu_bytes = active * w13_bytes                                            # packed gate/up codes + scales
        achieved = gu_bytes / (kinds["gate_up"]["us_per_launch"] * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": traffic[0] if traffic else None,
                "traffic_unit": "bytes per launch (ncu dram read + write)",
                "traffic_source": ("one ncu capture of %s on %s" % traffic[1:]) if traffic else None,
                "kernel": "gate_up (pair_gateup_wide_kernel)" if T * shape.top_k <= 24 else "gate_up (stream_gemm_kernel<1,true,1>)",
                "bytes_per_launch": gu_bytes, "peak_source": peaks["source"] + " copy rate, burst",
                "whole_step": {"achieved": step_gbs, "bytes_per_step": active_all * bpe, "frac": step_gbs / peaks["hbm_gbs"]}}
    if not identity:
        roof["note"] = ("C < E: the timed launches include resolution and the waves' miss traffic, so this fraction is not a "
                        "kernel figure; the workload is bound by the host link")
    res.update({"roofline": roof, "kernel_us": kinds, "active_experts_per_step": active_all,
                "packed_gb_per_s_whole_step": step_gbs, "tflops_whole_step": step_tflops, "bytes_per_expert": bpe})

    extra = {}
    if not identity:
        st = cache.stats(0)
        extra = {"hit_rate": st["hits"] / max(st["lookups"], 1), "h2d_expert_bytes_per_token":
                 st["h2d_bytes"] / max(st["forwards"] * T, 1), "waves_per_step": st["waves"] / max(st["forwards"], 1)}
        # the H2D link is the roofline of this workload: miss-traffic busy time and rate vs a plain pinned copy
        n_c = min(K, 100)
        cache.profile_enable(True)
        b0 = cache.stats(0)["h2d_bytes"]
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            c0.record(stream)
            for j in range(n_c):                              # steps spread evenly over the timed range (all alpha blocks)
                i = W + j * max(K // n_c, 1)
                step(i, outs[i & 1])
            c1.record(stream)
        stream.synchronize()
        copy_ms, _ = cache.profile_read(4)
        gemm_ms = cache.profile_read(1)[0] + cache.profile_read(2)[0]
        fetch_ms, fetch_with_gemm_ms = cache.profile_overlap()   # device timestamps of the brackets on both streams
        wall_ms = c0.elapsed_time(c1)
        moved = cache.stats(0)["h2d_bytes"] - b0
        cache.profile_enable(False)
        big = banks[0][:32]                                  # 104 MB of the pinned bank
        dst = torch.empty_like(big, device=dev)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dst.copy_(big, non_blocking=True)
        torch.cuda.synchronize()
        p0.record()
        dst.copy_(big, non_blocking=True)
        p1.record()
        torch.cuda.synchronize()
        ceiling = big.numel() / p0.elapsed_time(p1) / 1e6
        rate = moved / max(copy_ms, 1e-9) / 1e6
        res["roofline_gemm_view"] = res.pop("roofline")      # not a kernel figure here: the step is bound by the host link
        res["roofline"] = {"bound": "host link", "achieved": rate, "peak": ceiling, "unit": "GB/s", "frac": rate / ceiling,
                           "kernel": "fetch_misses_kernel (reads of the mapped pinned bank)" if args.miss_path == "device"
                           else "host-issued cudaMemcpyAsync per miss",
                           "whole_step_frac": (moved / n_c) / (ms_step * 1e-3) / 1e9 / ceiling,
                           "miss_traffic_busy_fraction": copy_ms / wall_ms, "gemm_kernels_busy_fraction": gemm_ms / wall_ms,
                           "fetch_time_overlapped_with_gemm_kernels": {"ms": fetch_with_gemm_ms, "of_fetch_ms": fetch_ms,
                                                                       "fraction": fetch_with_gemm_ms / max(fetch_ms, 1e-9),
                                                                       "of_gemm_time": fetch_with_gemm_ms / max(gemm_ms, 1e-9)},
                           "h2d_bytes_per_step": moved / n_c,
                           "peak_source": "one 104 MB pinned-host-to-device copy, measured in this run"}
        res["kernel_us"] = {"note": "C < E: single-kind launches still carry resolution and miss traffic; see roofline"}
        del dst
    res["extra"] = extra

    if full:
        # ---- end to end: host buffers in, host buffer out, copies inside the timed region
        n_e2e = 4 if args.profile_run else min(max(K, 100), 300)
        n_host = 8 if identity else min(n_sets, 128)
        pick = [(j * n_sets) // n_host for j in range(n_host)]
        h_h = [hs[j].cpu().pin_memory() for j in pick]
        h_i = [ids[j].cpu().pin_memory() for j in pick]
        h_w = [ws[j].cpu().pin_memory() for j in pick]
        h_out = torch.empty_like(h_h[0]).pin_memory()

        # the library's host-buffer entry point: inputs in host memory, result in host memory, synchronous; one call per
        # step (it stages the three inputs, copies them to the device in one copy, runs the layer and waits; tiny batches
        # replay a graph recorded per (layer, T), small results are written straight into pinned host memory, large
        # page-locked tensors are used in place)
        def e2e_step(i):
            j = i % len(h_h)
            cache.forward_host(i % L, h_h[j], h_i[j], h_w[j], out=h_out, stream=stream)

        for i in range(max(3, 2 * L)):                      # every layer's graph (tiny batches) is recorded before the timed calls
            e2e_step(i)
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            e2e_step(i)
        dt = time.perf_counter() - t0
        dt = max_over_ranks(dt, world, dev)
        h2d = h_h[0].numel() * 2 + h_i[0].numel() * 4 + h_w[0].numel() * 4
        res["e2e"] = {"value": world * n_e2e * T / dt, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                      "d2h_bytes_per_step": int(h_out.numel() * 2), "steps": n_e2e,
                      "mode": "exmoe_moe_forward_host: host tensors in and out, one synchronous call per step"}
        res["inputs"] = (hs, ids, ws)
    res["status"] = cache.status()
    cache.close()
    del cache
    torch.cuda.empty_cache()
    return res


def leg_summary(r):
    """The part of a leg that goes under config.<name> of the main line."""
    out = {"workload": r["desc"], "tokens_per_step": r["T"], "slots": r["C"], "steps": r["K"], "warmup": r["W"],
           "value": r["value"], "unit": UNIT, "ms_per_step": r["ms_per_step"], "repetitions": r["repetitions"],
           "timing": "CUDA graph replay of all steps" if r["graphable"] else "host-driven loop (one plan read-back per step)",
           "active_experts_per_step": r["active_experts_per_step"], "packed_gb_per_s_whole_step": r["packed_gb_per_s_whole_step"],
           "tflops_whole_step": r["tflops_whole_step"], "kernel_us": r["kernel_us"], "roofline": r["roofline"],
           "gpu_launches": r["launches"], "clocks": r["clocks"], "status": r["status"]}
    out.update(r["extra"])
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="decode", choices=sorted(WORKLOADS) + ["stack"])
    ap.add_argument("--alpha", type=float, default=None,
                    help="Zipf skew: overrides the workload's alpha (stack workload: default 0.5)")
    ap.add_argument("--miss-path", default="device", choices=["host", "device"],
                    help="C < E workloads: the device-initiated fetch kernel (the library's default) or host-issued miss copies")
    ap.add_argument("--prefetch", action="store_true",
                    help="stack workload, C < E: guess layer l+1's experts by routing layer l's input with layer l+1's "
                         "router and prefetch them on a side stream while layer l runs (exmoe_cache_prefetch)")
    ap.add_argument("--slots", type=int, default=0, help="override the workload's resident slots per layer")
    ap.add_argument("--tokens", type=int, default=0, help="override the workload's tokens per step")
    ap.add_argument("--cpu-budget", type=float, default=15.0, help="seconds of CPU oracle work for cpu_baseline")
    ap.add_argument("--layers", type=int, default=0, help="layer banks to rotate over (0 = the workload's default)")
    ap.add_argument("--no-extra-legs", action="store_true",
                    help="decode workload: skip the short prefill (config 4) and offload (config 3) legs")
    ap.add_argument("--profile-run", action="store_true",
                    help="for captures under a profiler: one repetition of one replay per timed region, no extra legs, no "
                         "CPU oracle leg, a short end-to-end loop (the printed numbers are then not bench values)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        args.steps_requested = args.steps
        if args.steps > 50:
            args.steps = 50
        args.warmup = min(args.warmup, 20)
        run_reference(args, rank, world)
        return

    import torch.distributed as dist
    from paper_2608_15383_b200 import binding, build
    if rank == 0:
        build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    binding.lib()

    if args.workload == "stack":
        rows = run_stack_sweep(args, dev, binding)
        if rank == 0:
            best = max(r["tokens_per_s"] for r in rows)
            print(json.dumps({"metric": "stack_tokens_per_s", "value": best, "unit": UNIT, "n_gpus": world,
                              "steps": args.steps, "warmup": args.warmup, "higher_is_better": True, "scaling": "weak",
                              "vs_baseline": None, "data": "synthetic", "dtype": "int4 weights x bf16 activations, fp32 accumulate",
                              "config": {"workload": "config5: 16-layer OLMoE-shaped MoE stack, decode batch x slot sweep, "
                                         "Zipf routing; the step includes the fused router kernel (Eq. 1) and the torch residual update between layers",
                                         "sweep": rows}}), flush=True)
        return
    shape = synth.OLMOE
    K, W = args.steps, max(args.warmup, 3)
    peaks = load_peaks()
    if args.profile_run:
        global MIN_REGION_MS, REPS
        MIN_REGION_MS, REPS = 0.0, 1
        args.no_extra_legs, args.cpu_budget = True, 0.0

    # ---- data: replicas only, every rank holds the same workload with its own seed offset
    seed0 = 2000 + 100000 * rank
    L = args.layers or WORKLOADS[args.workload][2]
    banks, w_cpu = build_banks(shape, L, seed0, dev, keep_layer0=(rank == 0))
    main_leg = run_leg(args.workload, args, shape, banks, dev, rank, local_rank, world, peaks, K, W, seed0, full=True)
    hs, ids, ws = main_leg.pop("inputs")
    T = main_leg["T"]

    legs = {}
    if args.workload == "decode" and not args.no_extra_legs and not (args.tokens or args.slots):
        # the other two parts of the metric, short: prefill TFLOP/s (config 4) and the offloaded decode (config 3)
        legs["prefill"] = leg_summary(run_leg("prefill", args, shape, banks, dev, rank, local_rank, world, peaks, 50, 3, seed0 + 7, full=False))
        legs["offload"] = leg_summary(run_leg("offload", args, shape, banks, dev, rank, local_rank, world, peaks, 100, 5, seed0 + 9, full=False))

    if rank == 0:
        cpu = oracle_leg(shape, T, w_cpu, hs, ids, ws, args.cpu_budget)
        bpe = main_leg["bytes_per_expert"]
        Lm = main_leg["L"]
        config = {"workload": main_leg["desc"], "tokens_per_step": T, "slots": main_leg["C"], "layers_rotated": Lm,
                  "l2": "inputs larger than L2: steps rotate over %d layer banks (%.2f GB packed)" % (Lm, Lm * 64 * bpe / 1e9)
                  if Lm > 1 else "single layer bank (%.0f MB packed) vs 126 MB L2" % (64 * bpe / 1e6),
                  "timing": ("CUDA graph replay of all steps" if main_leg["graphable"] else "host-driven loop (one plan read-back per step)") +
                            "; the K-step region is repeated back to back (see repetitions), the median repetition is reported",
                  "repetitions": main_leg["repetitions"],
                  "active_experts_per_step": main_leg["active_experts_per_step"],
                  "packed_gb_per_s_whole_step": main_leg["packed_gb_per_s_whole_step"],
                  "tflops_whole_step": main_leg["tflops_whole_step"],
                  "kernel_us": main_leg["kernel_us"], "parallelism": "replicas only (no collective)", "status": main_leg["status"],
                  "pack": dict(PACK_STATS), **main_leg["extra"], **legs}
        line = {"metric": METRIC, "value": main_leg["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": main_leg["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "int4 weights x bf16 activations, fp32 accumulate", "data": "synthetic",
                "config": config, "roofline": main_leg["roofline"], "cpu_baseline": cpu, "e2e": main_leg["e2e"],
                "gpu_launches": main_leg["launches"], "clocks": main_leg["clocks"]}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
