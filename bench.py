#!/usr/bin/env python
"""Throughput benchmark of the DynaMo quantized-MoE hot path on B200.

One step = one whole pass of the hot path (route -> permute -> mixed-precision grouped SwiGLU FFN
with the significant-channel correction -> weighted combine) over one synthetic batch of T tokens
through one MoE layer, via the C-ABI call ``dynamo_moe_forward``.  Steps rotate over several
independently generated layers so that the packed weights of a step always come from HBM (the
rotating set is far larger than L2).

Prints ONE JSON line.  The default run (decode workload) carries the whole metric: the headline is decode at
T = 64; ``extra`` holds T = 1, 8, 32, 64 with the HBM roofline of the gate/up launch each, the prefill workload
(T = 4096) with its tensor roofline, and ``switch`` the runtime channel switch on a 16-layer stack.
``--impl reference`` times the CPU oracle instead (a deliberately plain float64 program; it is a reported
baseline, not a target).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_21135_b200 import workloads as wl  # noqa: E402

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            j = json.load(open(p))
            return float(j["hbm_gbs"]), float(j.get("bf16_tflops_sustained", j.get("bf16_tflops", 1590.0))), "measured"
        except Exception:
            pass
    return 6650.0, 1590.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.idx = device_index
        self.proc = None
        self.path = os.path.join("/tmp", f"dynamo_clocks_{os.getpid()}.csv")

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.idx)], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                mx.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                 parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def device_layer_weights(cfg, layer, device):
    """The weight recipe of workloads.expert_weights (N(0, 0.02^2), each routed expert's outlier input channels
    x20 in W_gate and W_up, rounded to bf16) drawn on the device: a 1.4-billion-weight layer takes the host cores
    ten seconds and the GPU a few milliseconds, and the timed runs need many layers.  Same distribution, other
    draws than the host recipe, which stays the one the parity tests and the CPU baseline use."""
    g = torch.Generator(device=device)
    g.manual_seed(wl.BASE_SEED * 1000 + cfg.config_id * 100 + layer)
    n, d, f = cfg.n_total, cfg.d_model, cfg.d_ff
    out = []
    for shape, outliers in (((n, f, d), True), ((n, f, d), True), ((n, d, f), False)):
        w = torch.empty(shape, dtype=torch.float32, device=device)
        w.normal_(0.0, 0.02, generator=g)
        if outliers:
            for e in range(cfg.n_experts):
                cols = torch.from_numpy(wl.outlier_channels(cfg, layer, e).astype(np.int64)).to(device)
                w[e][:, cols] *= 20.0
        out.append(w.to(torch.bfloat16))
        del w
    return tuple(out)


def build_layers(cfg, n_layers, max_tokens, device, tc_min_rows=None, down_side=0, host_recipe=False):
    """Generate, upload and pack ``n_layers`` independent layers; they share one workspace."""
    from paper_2503_21135_b200 import binding

    layers, meta, ws = [], [], None
    for l in range(n_layers):
        if host_recipe:
            wg, wu, wd = wl.layer_weights(cfg, l, threads=min(16, os.cpu_count() or 8))
        else:
            wg, wu, wd = device_layer_weights(cfg, l, device)
        bits = wl.bits_assignment(cfg, l)
        pool = wl.cache_pool(cfg, l)
        sets = wl.initial_sig_sets(cfg, pool, l)
        layer = binding.DynamoLayer.from_config(cfg, max_tokens=max_tokens, workspace=ws, device=device)
        layer.pack_experts(wg.to(device), wu.to(device), wd.to(device), bits, pool)
        layer.set_channel_switch(sets)
        if down_side > 0:  # significant hidden units on the d_ff side: 2 * down_side cached, down_side significant
            pool_d = wl.cache_pool_down(cfg, 2 * down_side, l)
            layer.pack_down_cache(wd.to(device), bits, pool_d, down_side)
            layer.set_channel_switch_down(wl.sig_sets_down(cfg, pool_d, down_side, l))
        if tc_min_rows is not None:
            layer.set_tc_min_rows(tc_min_rows)
        torch.cuda.synchronize()
        ws = layer.workspace
        layers.append(layer)
        meta.append(dict(bits=bits, pool=pool, sets=sets))
        del wg, wu, wd
    return layers, meta


def active_experts(cfg, logits: torch.Tensor):
    idx = torch.topk(logits, cfg.top_k, dim=1).indices
    return sorted(set(int(e) for e in idx.flatten().tolist())) + list(range(cfg.n_experts, cfg.n_total))


def time_steps(fn, steps, dist_barrier):
    """Time ``steps`` calls of fn(i) with CUDA events on the current stream; returns ms total."""
    dist_barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    dist_barrier()
    return e0.elapsed_time(e1)


# dram__bytes_read.sum + dram__bytes_write.sum of one gate/up launch, from the ncu captures summarised
# under profiles/ (decode shape, layer 0); None where no capture of that launch exists.
NCU_TRAFFIC_BYTES = {("decode", 8): 493.8e6 + 3.8e6, ("decode", 64): 497.4e6 + 10.2e6}


def kernel_times(layers, step_fn, steps):
    """Average device time of the gate/up and the down FFN launch, measured live with CUDA events that
    the library records on the launching stream around those launches (a second pass over the steps)."""
    n = min(steps, 200)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(n)]
    for trio in evs:
        for e in trio:
            e.record()                      # creates the underlying handles
    torch.cuda.synchronize()
    for i in range(n):
        layer = layers[i % len(layers)]
        layer.set_profile_events(evs[i])
        step_fn(i)
        layer.set_profile_events(None)
    torch.cuda.synchronize()
    gu = [evs[i][0].elapsed_time(evs[i][1]) for i in range(n)]
    dn = [evs[i][1].elapsed_time(evs[i][2]) for i in range(n)]
    return float(np.mean(gu)), float(np.mean(dn))


def slowest_rank(times_ms, world, device):
    """Replicas only: ranks exchange nothing but their timings; a job is as slow as its slowest rank."""
    if world <= 1:
        return list(times_ms)
    t = torch.tensor(list(times_ms), device=device, dtype=torch.float64)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(tokens_per_rank, world, ms_per_step):
    """Whole-job tokens/s: every rank pushes its own batch through its own replica (weak scaling)."""
    return world * tokens_per_rank / (ms_per_step / 1e3)


def time_workload(cfg, layers, meta, T, steps, warmup, rank, world, device, barrier, hbm_peak, tensor_peak, peak_kind,
                  want_clocks=True):
    """Time `steps` forwards of T tokens rotating over `layers`; returns a result dict with throughput, the live
    per-launch times of the two FFN launches and the roofline block of the dominant (gate/up) launch."""
    from paper_2503_21135_b200 import binding

    n_layers = len(layers)
    xs = [wl.activations(cfg, T, l, step=0).to(device) for l in range(n_layers)]
    lgs_cpu = [wl.router_logits(cfg, T, l, step=0) for l in range(n_layers)]
    lgs = [t.to(device) for t in lgs_cpu]
    ys = [torch.empty((T, cfg.d_model), dtype=torch.float32, device=device) for _ in range(n_layers)]

    def step(i):
        l = i % n_layers
        layers[l].forward(xs[l], lgs[l], binding.F32, y=ys[l])

    sampler = ClockSampler(torch.cuda.current_device()) if want_clocks and rank == 0 else None
    if sampler:
        sampler.start()
        t_end = time.time() + 0.6        # keep the GPU under load while the sampler comes up
        while time.time() < t_end:
            for i in range(20):
                step(i)
            torch.cuda.synchronize()
    for i in range(max(warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    l0 = sum(l.kernel_launches() for l in layers)
    ms = time_steps(step, steps, barrier)
    launches = sum(l.kernel_launches() for l in layers) - l0
    gu_ms, dn_ms = kernel_times(layers, step, max(steps, 50))
    clocks = sampler.stop() if sampler else None
    for l in layers:
        assert l.poll_status() == 0, "device status word set (expired wait or clamped activation)"
    (ms_step,) = slowest_rank([ms / steps], world, device)
    res = {"tokens": T, "steps": steps, "ms_per_step": ms_step, "tokens_per_s": job_throughput(T, world, ms_step),
           "gpu_launches": launches, "gateup_ms": gu_ms, "down_ms": dn_ms, "clocks": clocks}
    d, f, G = cfg.d_model, cfg.d_ff, cfg.group_size
    pick = [i % n_layers for i in range(steps)]
    if T >= 512:
        # prefill-sized: the gate/up tcgen05 launch is bound by the tensor cores.  Algorithmic flops of the launch =
        # 2 * 2 * d * f per (token, expert) row + 2 * 2 * f * |S_e| for rows of switchable experts.
        fl = []
        for i in range(n_layers):
            idx = torch.topk(lgs_cpu[i], cfg.top_k, dim=1).indices.flatten()
            cnt = torch.bincount(idx, minlength=cfg.n_experts).tolist() + [T] * cfg.n_shared
            fl.append(sum(c * (4 * d * f + (4 * f * len(meta[i]["sets"][e])
                                            if e < cfg.n_experts and int(meta[i]["bits"][e]) < 8 else 0))
                          for e, c in enumerate(cnt)))
        gu_flops = float(np.mean([fl[i] for i in pick]))
        achieved = gu_flops / (gu_ms / 1e3) / 1e12
        burst = measured_burst()
        res["roofline"] = {"bound": "tensor", "achieved": achieved, "peak": tensor_peak, "unit": "TFLOP/s",
                           "frac": achieved / tensor_peak, "traffic": None,
                           "peak_kind": peak_kind + " (sustained fp16/bf16 cuBLAS; the kernel runs inside a long step)",
                           "frac_of_burst_peak": achieved / burst if burst else None, "burst_peak": burst,
                           "frac_of_nominal_2250": achieved / 2250.0,
                           "kernel": "ffn_tc2_kernel<gate/up> (+ streaming kernel for experts of <= 32 rows)",
                           "algorithmic_flops_per_launch": gu_flops, "avg_launch_ms": gu_ms,
                           "down_launch": {"achieved": gu_flops / 2 / (dn_ms / 1e3) / 1e12, "avg_launch_ms": dn_ms},
                           "whole_step": {"achieved": 1.5 * gu_flops / (ms_step / 1e3) / 1e12,
                                          "frac": 1.5 * gu_flops / (ms_step / 1e3) / 1e12 / tensor_peak,
                                          "frac_of_nominal_2250": 1.5 * gu_flops / (ms_step / 1e3) / 1e12 / 2250.0}}
    else:
        # decode-sized: HBM-bound on the packed bytes (+ significant tiles) of the experts a step activates
        gu_b, dn_b = [], []
        for i in range(n_layers):
            act = active_experts(cfg, lgs_cpu[i])
            tot = sum(layers[i].stream_bytes(e) for e in act)
            dn = sum(d * f * int(meta[i]["bits"][e]) // 8 + d * f // G * 4 for e in act)
            gu_b.append(tot - dn)
            dn_b.append(dn)
        gu_bytes = float(np.mean([gu_b[i] for i in pick]))
        dn_bytes = float(np.mean([dn_b[i] for i in pick]))
        achieved = gu_bytes / (gu_ms / 1e3) / 1e9
        step_gbs = (gu_bytes + dn_bytes) / (ms_step / 1e3) / 1e9
        res["roofline"] = {"bound": "hbm", "achieved": achieved, "peak": hbm_peak, "unit": "GB/s",
                           "frac": achieved / hbm_peak, "traffic": NCU_TRAFFIC_BYTES.get((cfg.name, T)),
                           "peak_kind": peak_kind, "frac_of_nominal_8000": achieved / 8000.0,
                           "kernel": "ffn_stream_kernel<gate/up>",
                           "algorithmic_bytes_per_launch": gu_bytes, "avg_launch_ms": gu_ms,
                           "down_launch": {"achieved": dn_bytes / (dn_ms / 1e3) / 1e9, "avg_launch_ms": dn_ms},
                           "whole_step": {"achieved": step_gbs, "frac": step_gbs / hbm_peak,
                                          "frac_of_nominal_8000": step_gbs / 8000.0}}
    return res, (xs, lgs_cpu)


def measured_burst():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(p))["bf16_tflops"])
    except Exception:
        return None


def run_ours(args, rank, world, device):
    from paper_2503_21135_b200 import binding, build

    build.build_library()
    binding.load()
    cfg = wl.CONFIGS[args.workload]
    T = args.tokens
    hbm_peak, tensor_peak, peak_kind = measured_peaks()
    full = args.workload == "decode" and not args.single   # the default run: the whole metric on one line

    def barrier():
        if world > 1:
            torch.distributed.barrier()

    n_layers = args.layers if not full else max(args.layers, 16 if not args.no_switch else args.layers)
    layers, meta = build_layers(cfg, n_layers, max(T, max(cfg.tokens)), device, args.tc_min_rows, args.down_side)
    rot = layers[:args.layers], meta[:args.layers]     # the layers a timed run rotates over (weights from HBM)
    common = dict(rank=rank, world=world, device=device, barrier=barrier, hbm_peak=hbm_peak, tensor_peak=tensor_peak,
                  peak_kind=peak_kind, want_clocks=not args.no_clocks)
    head, _ = time_workload(cfg, rot[0], rot[1], T, args.steps, args.warmup, **common)
    extra = {}
    sweep_T = [t for t in cfg.tokens if t != T] if (full or args.sweep) else []
    for Tcur in sweep_T:
        extra[str(Tcur)], _ = time_workload(cfg, rot[0], rot[1], Tcur, max(args.steps, 200), args.warmup, **common)
    extra[str(T)] = head

    router = None
    if args.router:
        # the same step with the router GEMM + top-k fused in front (scores from synthetic router weights, so the
        # routing differs from the logits-input run above: compare times at token counts where every expert is active)
        nl = len(rot[0])
        wrd = [tuple(t.to(device) for t in wl.router_weights(cfg, l)) for l in range(nl)]
        xs = [wl.activations(cfg, T, l, step=0).to(device) for l in range(nl)]

        def step_router(i):
            l = i % nl
            rot[0][l].forward_router(xs[l], wrd[l][0], wrd[l][1], binding.F32)

        for i in range(max(args.warmup, 3)):
            step_router(i)
        ms_r = time_steps(step_router, args.steps, barrier)
        router = {"ms_per_step_with_router_gemm": ms_r / args.steps, "tokens_per_s": world * T / (ms_r / args.steps / 1e3)}

    # end-to-end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    nl = len(rot[0])
    xh = [wl.activations(cfg, T, l, step=0).pin_memory() for l in range(nl)]
    lh = [wl.router_logits(cfg, T, l, step=0).pin_memory() for l in range(nl)]
    yh = [torch.empty((T, cfg.d_model), dtype=torch.float32).pin_memory() for _ in range(nl)]

    def step_host(i):
        l = i % nl
        rot[0][l].forward_host(xh[l], lh[l], yh[l], binding.F32)

    for i in range(3):
        step_host(i)
    ms_e2e = time_steps(step_host, args.steps, barrier)
    (ms_e2e,) = slowest_rank([ms_e2e / args.steps], world, device)

    out = {
        "metric": METRIC, "value": head["tokens_per_s"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None,
        "dtype": "f16 (integer codes x fp16 activations, fp32 accumulate)", "data": "synthetic (weights drawn on the device from the recipe's distribution, activations and logits from the seeded host recipe)",
        "config": {"workload": f"{cfg.name}: d_model={cfg.d_model} d_ff={cfg.d_ff} E={cfg.n_experts} top{cfg.top_k} "
                               f"G={cfg.group_size} S={cfg.max_sig} T={T}",
                   "tokens": T, "layers_rotated": len(rot[0]), "l2": "inputs larger than L2 (rotating layer arenas)",
                   "parallelism": "replicas only" if world > 1 else "single gpu",
                   **({"down_side_significant": args.down_side} if args.down_side else {})},
        "e2e": {"value": job_throughput(T, world, ms_e2e), "unit": UNIT,
                "h2d_bytes_per_step": T * cfg.d_model * 2 + T * cfg.n_experts * 4,
                "d2h_bytes_per_step": T * cfg.d_model * 4},
        "gpu_launches": head["gpu_launches"],
        "clocks": head["clocks"],
        "roofline": head["roofline"],
    }
    if router is not None:
        out["router"] = router
    if cfg.n_experts == 8 and cfg.d_model == 4096 and not args.no_switch:
        out["switch"] = measure_switch(layers, meta, cfg, device)
    del layers, rot
    torch.cuda.empty_cache()
    if full and not args.no_prefill:
        # the prefill half of the metric: config 3 (4096 tokens, Zipf-skewed router), its own layers and roofline
        pcfg = wl.CONFIGS["prefill"]
        pT = max(pcfg.tokens)
        players, pmeta = build_layers(pcfg, 2, pT, device, args.tc_min_rows, 0)
        pres, _ = time_workload(pcfg, players, pmeta, pT, max(args.steps, 50), args.warmup, **common)
        pres["workload"] = (f"{pcfg.name}: d_model={pcfg.d_model} d_ff={pcfg.d_ff} E={pcfg.n_experts} top{pcfg.top_k} "
                            f"G={pcfg.group_size} S={pcfg.max_sig} T={pT}, 2 layers rotated")
        extra[f"prefill_{pT}"] = pres
        del players
        torch.cuda.empty_cache()
    out["extra"] = extra
    if rank == 0 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(cfg, T, args.cpu_tokens)
    return out


def measure_switch(layers, meta, cfg, device, T=16, events=8, steps_between=8):
    """Runtime channel switch on the stack of layers at hand (config 5 recipe: decode batch 16, every 8 steps
    25 % of each expert's significant channels are swapped for other cached channels): steady-state step time,
    latency of one whole switch event (all layers, one call) on the device and on the host, and its share of a step."""
    from paper_2503_21135_b200 import binding

    n = len(layers)
    xs = [wl.activations(cfg, T, l, step=1).to(device) for l in range(n)]
    lgs = [wl.router_logits(cfg, T, l, step=1).to(device) for l in range(n)]
    ys = [torch.empty((T, cfg.d_model), dtype=torch.float32, device=device) for _ in range(n)]

    def stack_step():
        for l in range(n):
            layers[l].forward(xs[l], lgs[l], binding.F32, y=ys[l])

    res = {}
    for mode_name, mode in (("select", binding.SWITCH_SELECT), ("requant", binding.SWITCH_REQUANT)):
        cur = [m["sets"] for m in meta]
        for l in layers:
            l.set_switch_mode(mode)
        binding.set_channel_switch_many(layers, cur)
        for _ in range(5):
            stack_step()
        torch.cuda.synchronize()
        dev_ms, host_ms, step_ms = [], [], []
        for ev in range(events):
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            new = [wl.switch_event(cfg, meta[l]["pool"], cur[l], l, ev) for l in range(n)]
            torch.cuda.synchronize()
            e0.record()
            for _ in range(steps_between):
                stack_step()
            e1.record()
            t0 = time.perf_counter()
            binding.set_channel_switch_many(layers, new)
            host_ms.append((time.perf_counter() - t0) * 1e3)
            e2.record()
            torch.cuda.synchronize()
            step_ms.append(e0.elapsed_time(e1) / steps_between)
            dev_ms.append(e1.elapsed_time(e2))
            cur = new
        for l in layers:
            l.set_switch_mode(binding.SWITCH_SELECT)
        binding.set_channel_switch_many(layers, [m["sets"] for m in meta])
        sm, dm, hm = float(np.median(step_ms)), float(np.median(dev_ms)), float(np.median(host_ms))
        res[mode_name] = {"layers": n, "tokens": T, "stack_step_ms": sm, "tokens_per_s": T / (sm / 1e3),
                          "switch_event_device_ms": dm, "switch_event_host_ms": hm,
                          "switch_fraction_of_step": dm / sm, "events": events}
    # device-side selection: statistics collected during the forwards, then per layer one call that ranks the cached
    # channels and rewrites the tables (it synchronises to bring the chosen sets back to the host mirror)
    for l in layers:
        l.set_stats_collection(True)
    for _ in range(3):
        stack_step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps_between):
        stack_step()
    e1.record()
    torch.cuda.synchronize()
    step_stats_ms = e0.elapsed_time(e1) / steps_between
    # the selection of all layers is enqueued without waiting (the chosen sets reach the host mirror later)
    e0.record()
    t0 = time.perf_counter()
    for l in layers:
        l.select_significant(cfg.max_sig, reset=True, wait=False)
    sel_host_ms = (time.perf_counter() - t0) * 1e3
    e1.record()
    torch.cuda.synchronize()
    sel_dev_ms = e0.elapsed_time(e1)
    for l in layers:
        l.sync_sets()
    for l in layers:
        l.set_stats_collection(False)
    binding.set_channel_switch_many(layers, [m["sets"] for m in meta])
    res["device_selection"] = {"layers": n, "tokens": T, "stack_step_ms_with_stats": step_stats_ms,
                               "select_all_layers_host_enqueue_ms": sel_host_ms,
                               "select_all_layers_device_ms": sel_dev_ms}
    return res


def cpu_baseline(cfg, T, n_tokens):
    """The oracle as it stands, timed on the host cores on a bounded sample of the same workload."""
    import oracle

    wg, wu, wd = wl.layer_weights(cfg, 0, threads=min(16, os.cpu_count() or 8))
    bits = wl.bits_assignment(cfg, 0)
    pool = wl.cache_pool(cfg, 0)
    sets = wl.initial_sig_sets(cfg, pool, 0)
    x, lg = wl.activations(cfg, T, 0, 0), wl.router_logits(cfg, T, 0, 0)
    n_tokens = min(n_tokens, T)
    idx, _ = oracle.route(lg.numpy(), cfg.top_k)
    need = sorted(set(int(e) for e in idx[:n_tokens].ravel())) + list(range(cfg.n_experts, cfg.n_total))
    ora = oracle.OracleLayer(oracle.as_u16(wg), oracle.as_u16(wu), oracle.as_u16(wd), bits, cfg.group_size,
                             cfg.n_experts, cfg.top_k, experts=need)
    ora.set_channel_switch(sets)
    t0 = time.perf_counter()
    ora.forward(oracle.as_u16(x), lg.numpy(), tokens=np.arange(n_tokens, dtype=np.int32))
    dt = time.perf_counter() - t0
    return {"value": n_tokens / dt, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"first {n_tokens} of {T} tokens of layer 0, quantization excluded, {dt:.2f} s"}


def run_reference(args, rank, world):
    if rank != 0:
        return None
    cfg = wl.CONFIGS[args.workload]
    T = args.tokens
    import oracle

    wg, wu, wd = wl.layer_weights(cfg, 0, threads=min(16, os.cpu_count() or 8))
    bits = wl.bits_assignment(cfg, 0)
    pool = wl.cache_pool(cfg, 0)
    sets = wl.initial_sig_sets(cfg, pool, 0)
    x, lg = wl.activations(cfg, T, 0, 0), wl.router_logits(cfg, T, 0, 0)
    n_tok = min(args.cpu_tokens, T)
    idx, _ = oracle.route(lg.numpy(), cfg.top_k)
    need = sorted(set(int(e) for e in idx[:n_tok].ravel())) + list(range(cfg.n_experts, cfg.n_total))
    ora = oracle.OracleLayer(oracle.as_u16(wg), oracle.as_u16(wu), oracle.as_u16(wd), bits, cfg.group_size,
                             cfg.n_experts, cfg.top_k, experts=need)
    ora.set_channel_switch(sets)
    toks = np.arange(n_tok, dtype=np.int32)
    steps, warm = min(args.steps, 3), min(args.warmup, 1)
    for _ in range(warm):
        ora.forward(oracle.as_u16(x), lg.numpy(), tokens=toks)
    t0 = time.perf_counter()
    for _ in range(steps):
        ora.forward(oracle.as_u16(x), lg.numpy(), tokens=toks)
    dt = (time.perf_counter() - t0) / steps
    value = n_tok / dt
    sample = f"each step = the first {n_tok} of {T} tokens of layer 0 (quantization excluded)"
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: d_model={cfg.d_model} d_ff={cfg.d_ff} E={cfg.n_experts} "
                                   f"top{cfg.top_k} G={cfg.group_size} S={cfg.max_sig} T={T}", "tokens": T},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: run the same command line as N local ranks under torchrun."""
    import socket

    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "replica-selftest"])
    ap.add_argument("--workload", default="decode", choices=list(wl.CONFIGS))
    ap.add_argument("--tokens", type=int, default=None, help="default: the workload's largest token count")
    ap.add_argument("--layers", type=int, default=None,
                    help="independent layers rotated over so that weights come from HBM (default 4; 16 for switch)")
    ap.add_argument("--no-switch", action="store_true", help="skip the runtime channel-switch measurement")
    ap.add_argument("--tc-min-rows", type=int, default=None,
                    help="experts with more rows than this take the tcgen05 kernel (0: streaming kernel only)")
    ap.add_argument("--router", action="store_true",
                    help="also time the forward with the router GEMM + top-k fused in front")
    ap.add_argument("--down-side", type=int, default=0,
                    help="also serve this many significant hidden units per expert at 8-bit on the d_ff side (W_down)")
    ap.add_argument("--sweep", action="store_true", help="also time the workload's other token counts")
    ap.add_argument("--single", action="store_true",
                    help="only the headline token count (the default decode run also reports T = 1, 8, 32, the prefill "
                         "workload and the 16-layer switch stack)")
    ap.add_argument("--no-prefill", action="store_true", help="skip the prefill entry of the default run")
    ap.add_argument("--no-clocks", action="store_true",
                    help="no clock sampling (and none of the load that precedes it): for short runs under a profiler")
    ap.add_argument("--cpu-tokens", type=int, default=16, help="tokens in the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.tokens is None:
        args.tokens = max(wl.CONFIGS[args.workload].tokens)
    if args.layers is None:
        args.layers = wl.CONFIGS[args.workload].n_layers if args.workload == "switch" else (2 if args.tokens >= 512 else 4)

    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        # no launcher around us: start one rank per GPU ourselves (independent replicas; see slowest_rank)
        raise SystemExit(spawn_ranks(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        out = run_reference(args, rank, world)
        if out is not None:
            print(json.dumps(out), flush=True)
        return
    if args.impl == "replica-selftest":
        # the N > 1 plumbing alone (rendezvous, MAX-reduction of timings, one line from rank 0), on gloo without a GPU
        torch.distributed.init_process_group("gloo")
        got = slowest_rank([1.0 + rank], world, torch.device("cpu"))
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
        if rank == 0:
            print(json.dumps({"impl": "replica-selftest", "n_gpus": world, "ms_per_step": got[0],
                              "value": job_throughput(1, world, got[0])}), flush=True)
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=device)
    out = run_ours(args, rank, world, device)
    if world > 1:
        torch.distributed.barrier()
        torch.distributed.destroy_process_group()
    if rank == 0:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
