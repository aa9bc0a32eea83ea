#!/usr/bin/env python
"""Benchmark of the FP8 transformer-block hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config c4|c3|c1]

One step = one pass of the whole hot path over one block of synthetic input: JIT quantize of every
activation / weight / gradient, the 12 FP8 GEMMs (forward, dgrad, wgrad of 4 projections), quantize of
Q/K/V/dO and FP8 attention forward + backward.  `value` = (GEMM + causal-attention FLOPs) / time in TFLOP/s
with inputs resident in HBM; `e2e` = the same with host->device copies of the BF16 inputs and device->host
copies of every output inside the timed region.  With N > 1 (torchrun) every rank runs an independent replica
(the path has no exchange step); the time is the max over ranks.

`--impl reference` times the CPU oracle (as it stands) on a bounded sample of the same workload.
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

METRIC = "FP8 GEMM + FP8 attention TFLOP/s (fwd+bwd) on 1 B200, % of dense FP8 peak"
UNIT = "TFLOP/s"
FP8_NOMINAL_TFLOPS = 4500.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_burst": d["bf16_tflops"], "bf16_sustained": d["bf16_tflops_sustained"], "hbm": d["hbm_gbs"],
                "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm": 6650.0, "source": "fallback"}


# ---------------------------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int, period: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
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
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake",
        }
        # the benign ones too, so that a clock below the maximum never comes without its reason
        for attr, name in (("nvmlClocksThrottleReasonGpuIdle", "gpu_idle"),
                           ("nvmlClocksThrottleReasonApplicationsClocksSetting", "applications_clocks_setting"),
                           ("nvmlClocksThrottleReasonSyncBoost", "sync_boost"),
                           ("nvmlClocksThrottleReasonDisplayClockSetting", "display_clock_setting")):
            if hasattr(nv, attr):
                names[getattr(nv, attr)] = name
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s), "sm_mhz_min": s[0] if s else None, "sm_mhz_max_seen": s[-1] if s else None}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ---------------------------------------------------------------------------------------------- oracle sample
def oracle_sample(cfg, reps: int = 1):
    """Runs the CPU oracle on a bounded sample of the workload; returns (flops, seconds, description)."""
    import numpy as np
    import oracle as o
    from paper_2505_20524_b200 import synth

    small = synth.BlockConfig(**{**cfg.__dict__})
    flops, secs = 0.0, 0.0
    desc = []
    if cfg.has_linears:
        T, N, K = cfg.linear_shapes()["qkv"]
        Ts = 512                                      # token slice of the QKV projection
        cols = synth.choose_columns(K, cfg.n_outlier_cols(K), cfg.seed, 100)
        x = synth.normal_bf16((Ts, K), cfg.seed, 0, 1.0, cols, cfg.act_outlier_factor)
        w = synth.normal_bf16((N, K), cfg.seed, 1, synth.W_STD)
        dy = synth.normal_bf16((Ts, N), cfg.seed, 8, synth.GRAD_STD)
        t0 = time.perf_counter()
        for _ in range(reps):
            x8, _, _, sx = o.quantize(x, o.E4M3)
            w8, _, _, sw = o.quantize(w, o.E4M3)
            dy8, _, _, sdy = o.quantize(dy, o.E5M2)
            rows = np.arange(128)
            o.linear_fwd(x8, w8, sx, sw, rows=rows)
            o.linear_dgrad(dy8, w8, sdy, sw, rows=rows)
            o.linear_wgrad(dy8, x8, sdy, sx, rows=rows)
        secs += time.perf_counter() - t0
        flops += reps * 2.0 * 128 * (N * K + N * K + Ts * K)
        desc.append(f"quantize + 128 output rows each of QKV fwd/dgrad/wgrad on a {Ts}-token slice")
    Na = min(1024, cfg.seq)
    q, k, v, do = synth.attention_inputs(small, seq=Na, batch=1)
    t0 = time.perf_counter()
    for _ in range(reps):
        q8, _, _, qi = o.quantize(q, o.E4M3)
        k8, _, _, ki = o.quantize(k, o.E4M3)
        v8, _, _, vi = o.quantize(v, o.E4M3)
        do8, _, _, doi = o.quantize(do, o.E5M2)
        G = cfg.n_q_heads // cfg.n_kv_heads
        p = o.attn_params(1, Na, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, kv_block=128, q_inv=qi, k_inv=ki,
                          v_inv=vi, do_inv=doi, ds_scale=4096.0)
        heads = [(0, h) for h in range(G)]
        O, lse, _ = o.attention_fwd(q8, k8, v8, p, heads=heads)
        Of = np.zeros((1, Na, cfg.n_q_heads, cfg.head_dim))
        Lf = np.zeros((1, cfg.n_q_heads, Na))
        Of[0, :, :G] = O.transpose(1, 0, 2)
        Lf[0, :G] = lse
        o.attention_bwd(q8, k8, v8, do8, Of, Lf, p, kv_heads=[(0, 0)])
    secs += time.perf_counter() - t0
    flops += reps * 3.5 * 2.0 * G * Na * Na * cfg.head_dim
    desc.append(f"attention fwd+bwd of one KV group ({G} heads) at seq {Na}")
    return flops, secs, "; ".join(desc), o.num_threads()


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(args.warmup):
        oracle_sample(cfg)
    flops, secs = 0.0, 0.0
    for _ in range(args.steps):
        f, s, desc, cores = oracle_sample(cfg)
        flops += f
        secs += s
    value = flops / secs / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name + " (bounded sample per step: " + desc + ")"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- other workloads
def quantize_sweep(peaks):
    """Workload c2: amax / cast / quantize on flat BF16 tensors of 2^20 .. 2^29 elements, N(0,1) with 1e-4 of the
    entries set to +-200.  `cold`: the calls walk a pool of tensors larger than twice the L2, so nothing is resident
    from the previous call; `warm`: the same tensor again and again (flagged: at the small sizes this is an L2 figure)."""
    import torch
    import paper_2505_20524_b200 as fp8
    out = []
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2)
    f32 = lambda v=0.0: torch.full((1,), float(v), dtype=torch.float32, device="cuda")
    for log2n in (20, 24, 27, 29):
        n = 1 << log2n
        nbuf = max(1, min(160, -(-(300 << 20) // (2 * n))))
        xs = []
        for _ in range(nbuf):
            x = torch.randn(n, device="cuda", generator=gen)
            hit = torch.rand(n, device="cuda", generator=gen) < 1e-4
            x = torch.where(hit, torch.where(x > 0, 200.0, -200.0), x).to(torch.bfloat16)
            xs.append(x)
            del hit
        q = torch.empty(n, dtype=torch.uint8, device="cuda")
        a, sc, si = f32(), f32(2.24), f32(1.0)
        ops = (("amax", 2, lambda x: fp8.fp8_amax(x, a)),
               ("cast_e4m3", 3, lambda x: fp8.fp8_cast(x, sc, fp8.E4M3, q)),
               ("cast_e5m2", 3, lambda x: fp8.fp8_cast(x, sc, fp8.E5M2, q)),
               ("quantize_e4m3", 5, lambda x: fp8.fp8_quantize(x, fp8.E4M3, q, None, a, sc, si)))
        row = {"elements": n, "pool_tensors": nbuf}
        for name, bpe, fn in ops:
            for mode in ("cold", "warm"):
                reps = max(8, nbuf) if mode == "cold" else 20
                for i in range(3):
                    fn(xs[i % nbuf])
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                e0.record()
                for i in range(reps):
                    fn(xs[i % nbuf] if mode == "cold" else xs[0])
                e1.record()
                torch.cuda.synchronize()
                gbs = bpe * n * reps / (e0.elapsed_time(e1) / 1e3) / 1e9
                row[f"{name}_{mode}_gbs"] = round(gbs, 1)
        row["quantize_cold_frac_of_measured_hbm"] = round(row["quantize_e4m3_cold_gbs"] / peaks["hbm"], 3)
        out.append(row)
        del xs, q
        torch.cuda.empty_cache()
    return {"workload": "c2: flat BF16 tensors, N(0,1) with 1e-4 of the entries +-200 (drawn on the device, seed 2)",
            "bytes_per_element": {"amax": 2, "cast": 3, "quantize": 5}, "hbm_gbs_measured": peaks["hbm"],
            "note": "warm = same tensor repeated (L2-resident below 2^26 elements); cold = pool of tensors > 2 x L2",
            "sizes": out}


def delayed_scaling_step(cfg, host, args, flops_step):
    """The same step under delayed scaling (Appendix E, the recipe the paper trains with): every tensor is cast in one
    pass under the scale of its abs-max history (length 1024), the pass records the new abs-max and the last block to
    finish a tensor updates history and scale for the next step (one launch per group of operands:
    fp8_quantize_delayed_multi).  Same inputs, same products and attention; the headline `value` stays the
    just-in-time form."""
    import torch
    from paper_2505_20524_b200.hotpath import BlockHotPath
    hp = BlockHotPath(cfg, attn_max_slack=args.attn_slack, scaling="delayed")
    hp.allocate(host)
    hp.calibrate_ds_scale()
    def run(step):
        for _ in range(3):
            step()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    ms = run(hp.step)
    ms_ov = run(hp.step_overlapped)
    out = {"ms_per_step": ms, "value": flops_step / ms / 1e9, "unit": UNIT, "quantize_gb_per_step": hp.quantize_bytes() / 1e9,
           "history_len": 1024, "launches_per_step": hp.launches_per_step(),
           "two_streams": {"ms_per_step": ms_ov, "value": flops_step / ms_ov / 1e9,
                           "what": "the cast passes on a side stream, in the shadow of the products"}}
    del hp
    torch.cuda.empty_cache()
    return out


def long_context_attention(peaks, steps=5):
    """Workload c5: causal FP8 attention forward + backward at B = 1, N = 16384, 32 heads x 128; Q/K/V N(0,1) with 1% of
    the (head, dim) columns x 40, dO N(0, 1e-3); drawn on the device (seed 5) and quantised by fp8_quantize."""
    import torch
    import paper_2505_20524_b200 as fp8
    B, N, H, d = 1, 16384, 32, 128
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    f32 = lambda v=0.0: torch.full((1,), float(v), dtype=torch.float32, device="cuda")
    t = {}
    for name, std, fmt in (("q", 1.0, fp8.E4M3), ("k", 1.0, fp8.E4M3), ("v", 1.0, fp8.E4M3), ("do", 1e-3, fp8.E5M2)):
        x = torch.randn((B, N, H, d), device="cuda", generator=gen) * std
        if name != "do":
            cols = torch.randperm(H * d, device="cuda", generator=gen)[:41]
            x.view(B, N, H * d)[:, :, cols] *= 40.0
        x = x.to(torch.bfloat16)
        q8 = torch.empty((B, N, H, d), dtype=torch.uint8, device="cuda")
        a, sc, si = f32(), f32(), f32()
        fp8.fp8_quantize(x, fmt, q8, None, a, sc, si)
        t[name] = (q8, si)
        del x
    O = torch.empty((B, N, H, d), dtype=torch.bfloat16, device="cuda")
    LSE = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(O), torch.empty_like(O), torch.empty_like(O)
    ws = torch.empty(fp8.fp8_attention_workspace_bytes(1, B, N, H, H, d), dtype=torch.uint8, device="cuda")
    s, dss, amax = d ** -0.5, f32(1.0), f32()
    fwd = lambda: fp8.fp8_attention_fwd(t["q"][0], t["k"][0], t["v"][0], t["q"][1], t["k"][1], t["v"][1], s, True, O,
                                        LSE, None)
    bwd = lambda: fp8.fp8_attention_bwd(t["q"][0], t["k"][0], t["v"][0], t["do"][0], O, LSE, t["q"][1], t["k"][1],
                                        t["v"][1], t["do"][1], s, dss, True, dq, dk, dv, ws, ds_amax=amax)
    fwd()
    bwd()                                        # calibration of the dS scale, delayed-scaling style
    fp8.fp8_scale(amax, fp8.E5M2, 0, dss, f32())
    res = {}
    for name, fn in (("fwd", fwd), ("bwd", bwd)):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        res[name] = e0.elapsed_time(e1) / steps
    fl = 2.0 * B * H * N * N * d
    tot = 3.5 * fl / (res["fwd"] + res["bwd"]) / 1e9
    return {"workload": "c5: B 1, N 16384, 32 heads x 128, causal; synthetic, drawn on the device (seed 5)",
            "fwd_ms": res["fwd"], "bwd_ms": res["bwd"], "fwd_tflops": fl / res["fwd"] / 1e9,
            "bwd_tflops": 2.5 * fl / res["bwd"] / 1e9, "fwd_bwd_tflops": tot,
            "fwd_bwd_frac_of_nominal_4500": tot / FP8_NOMINAL_TFLOPS,
            "fwd_bwd_frac_of_2x_burst": tot / (2.0 * peaks["bf16_burst"]), "steps": steps,
            "l2": "operands (4 x 67 MB) and outputs exceed the L2 together; no flush", "device_status": fp8.fp8_device_status()}


# ---------------------------------------------------------------------------------------------- our arm
def max_over_ranks(ms_local: float, world: int, device=None) -> float:
    """Device time of the slowest rank (every rank gets the same number)."""
    if world <= 1:
        return float(ms_local)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tflops(world: int, flops_per_step: float, steps: int, ms_total: float) -> float:
    """Whole-job throughput: every rank runs its own replica of the step (weak scaling)."""
    return world * flops_per_step * steps / (ms_total / 1e3) / 1e12


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    import paper_2505_20524_b200 as fp8
    from paper_2505_20524_b200.hotpath import BlockHotPath

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    fp8.binding.load()

    def barrier():
        if world > 1:
            dist.barrier()

    hp = BlockHotPath(cfg, dev, attn_max_slack=args.attn_slack)
    host = hp.generate_host_inputs()
    hp.allocate()
    hp.calibrate_ds_scale()
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        hp.step()
    torch.cuda.synchronize()

    # ---- device-resident timing (inputs already in HBM)
    sampler = ClockSampler(physical_gpu_index(local))
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        hp.step(time_gemms=True)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, dev)
    status = fp8.fp8_device_status()
    if status != 0:
        raise SystemExit(f"device status {status}: a bounded wait expired inside a kernel")

    flops_step = hp.gemm_flops() + hp.attention_flops()
    value = job_tflops(world, flops_step, args.steps, ms_total)

    graph_info = None
    if args.graph:
        # the same step submitted once per iteration: what is left of the step time when launch overhead is gone
        g = hp.capture_graph()
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        for _ in range(args.steps):
            g.replay()
        g1.record()
        torch.cuda.synchronize()
        barrier()
        g_ms = max_over_ranks(g0.elapsed_time(g1), world, dev)
        if fp8.fp8_device_status() != 0:
            raise SystemExit("device status: a bounded wait expired inside a kernel (graph replay)")
        graph_info = {"ms_per_step": g_ms / args.steps, "value": job_tflops(world, flops_step, args.steps, g_ms),
                      "unit": UNIT}

    # ---- dominant kernel: the FP8 GEMM; duration from the events recorded around each launch
    gemm_ms = sum(a.elapsed_time(b) for evs in hp.gemm_events for a, b in evs)
    n_gemm = sum(len(evs) for evs in hp.gemm_events)
    gemm_tflops = hp.gemm_flops() * args.steps / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else None
    peaks = measured_peaks()
    # Which measured peak the in-step rate is compared with.  FP8 is nominally 2x the BF16 rate, so the denominators
    # are 2 x the measured BF16 GEMM figures.  The sustained figure was taken over seconds at a power-capped clock;
    # a timed region shorter than a second that ran at (nearly) the maximum SM clock is a burst, and is compared
    # with the burst figure.  All three fractions are carried; `frac` is the one the rule picks.
    region_s = ms_total / 1e3
    clk_ok = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and
                  clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    use_burst = region_s < 1.0 or clk_ok
    fp8_peak = 2.0 * (peaks["bf16_burst"] if use_burst else peaks["bf16_sustained"])
    roofline = None
    if gemm_tflops is not None:
        traffic = GEMM_DRAM_CAPTURE.get(cfg.name)
        roofline = {
            "bound": "tensor", "kernel": "gemm_fp8_pair_kernel", "achieved": gemm_tflops, "peak": fp8_peak,
            "unit": "TFLOP/s", "frac": gemm_tflops / fp8_peak,
            "traffic": traffic["bytes_per_launch"] if traffic else None,
            "traffic_source": traffic["source"] if traffic else None,
            "peak_source": (f"2 x bf16_tflops{'' if use_burst else '_sustained'} ({peaks['source']}); rule: burst figure "
                            f"when the timed region is < 1 s or the sampled SM clock stays within 3% of its maximum "
                            f"(region {region_s:.2f} s, median clock {clocks.get('sm_mhz')} MHz), else sustained"),
            "launches": n_gemm, "avg_launch_ms": gemm_ms / max(n_gemm, 1),
            "flops_per_launch": hp.gemm_flops() / 12.0,
            "frac_vs_2x_burst": gemm_tflops / (2.0 * peaks["bf16_burst"]),
            "frac_vs_2x_sustained": gemm_tflops / (2.0 * peaks["bf16_sustained"]),
            "frac_of_nominal_4500": gemm_tflops / FP8_NOMINAL_TFLOPS,
        }

    # ---- the other parts of the step, from their own events: attention forward / backward and the quantize groups
    attention, quantize = None, None
    if hp.attn_events and hp.attn_events[0]:
        f_ms = sum(evs[0][0].elapsed_time(evs[0][1]) for evs in hp.attn_events) / args.steps
        b_ms = sum(evs[1][0].elapsed_time(evs[1][1]) for evs in hp.attn_events) / args.steps
        fwd_fl = hp.attention_flops() / 3.5
        attention = {"fwd_ms": f_ms, "bwd_ms": b_ms, "fwd_tflops": fwd_fl / f_ms / 1e9, "bwd_tflops": 2.5 * fwd_fl / b_ms / 1e9,
                     "fwd_frac_of_nominal_4500": fwd_fl / f_ms / 1e9 / FP8_NOMINAL_TFLOPS,
                     "bwd_frac_of_nominal_4500": 2.5 * fwd_fl / b_ms / 1e9 / FP8_NOMINAL_TFLOPS,
                     "fwd_bwd_tflops": 3.5 * fwd_fl / (f_ms + b_ms) / 1e9,
                     "fwd_bwd_frac_of_2x_burst": 3.5 * fwd_fl / (f_ms + b_ms) / 1e9 / (2.0 * peaks["bf16_burst"])}
    if hp.quant_events and hp.quant_events[0]:
        q_ms = sum(a.elapsed_time(b) for evs in hp.quant_events for a, b in evs) / args.steps
        gbs = hp.quantize_bytes() / q_ms / 1e6
        quantize = {"ms_per_step": q_ms, "gb_per_step": hp.quantize_bytes() / 1e9, "gbs": gbs,
                    "frac_of_measured_hbm": gbs / peaks["hbm"], "hbm_gbs": peaks["hbm"], "peak_source": peaks["source"]}

    # ---- end to end: pinned host inputs -> device, step, every output -> pinned host
    ins, outs = hp.input_tensors(), hp.output_tensors()
    h_in = [torch.from_numpy(host[n].view("int16")).view(torch.bfloat16).pin_memory() for n, _ in ins]
    h_out = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for _, t in outs]
    h2d = sum(t.numel() * t.element_size() for t in h_in)
    d2h = sum(t.numel() * t.element_size() for t in h_out)

    hin = {n: h for (n, _), h in zip(ins, h_in)}
    hout = {n: h for (n, _), h in zip(outs, h_out)}

    # through the C ABI's host-buffer entry points (one call per projection and one for the attention, each on its
    # own device workspace; the library pipelines uploads, kernels and downloads on its three streams)
    def e2e_step():
        hp.step_host_abi(hin, hout)

    e2e_steps = max(1, min(args.steps, 10))
    e2e_step()
    fp8.fp8_host_sync()
    torch.cuda.synchronize()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()               # consecutive steps overlap: uploads of one under the downloads of the last
    fp8.fp8_host_sync()          # the timed region ends when the last output is in host memory (a host wait)
    e1.record()
    torch.cuda.synchronize()
    barrier()
    e2e_value = job_tflops(world, flops_step, e2e_steps, max_over_ranks(e0.elapsed_time(e1), world, dev))

    # the same region with the copies and the device-pointer calls issued from the binding on torch streams
    hp.step_host(hin, hout, wait=False)
    hp.finish_host()
    torch.cuda.synchronize()
    barrier()
    e0.record()
    for _ in range(e2e_steps):
        hp.step_host(hin, hout, wait=False)
    hp.finish_host()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    e2e_binding_value = job_tflops(world, flops_step, e2e_steps, max_over_ranks(e0.elapsed_time(e1), world, dev))

    cpu_baseline = None
    if rank == 0 and world == 1:
        f, s, desc, cores = oracle_sample(cfg, reps=1)
        reps = int(min(16, max(1, round(15.0 / max(s, 1e-3)))))      # aim at 10-30 s of CPU work
        if reps > 1:
            f, s, desc, cores = oracle_sample(cfg, reps=reps)
        cpu_baseline = {"value": f / s / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                        "sample": f"{reps} x ({desc})", "seconds": s}

    acct = {"launches": hp.launches_per_step() * args.steps, "gemm_tflop": hp.gemm_flops() / 1e12,
            "attn_tflop": hp.attention_flops() / 1e12, "quant_gb": hp.quantize_bytes() / 1e9}
    c2, c5, delayed, two_streams = None, None, None, None
    if rank == 0 and world == 1 and not args.no_extra and cfg.name == "c4":
        # the same step with its quantize calls on a side stream (same kernels, same bits; the headline stays the
        # one-stream step, whose per-kernel events feed the roofline)
        for _ in range(3):
            hp.step_overlapped()
        torch.cuda.synchronize()
        e0.record()
        hp.gemm_events = []
        for _ in range(args.steps):
            hp.step_overlapped(time_gemms=True)
        e1.record()
        torch.cuda.synchronize()
        ms_ov = e0.elapsed_time(e1) / args.steps
        gemm_ms_ov = sum(a.elapsed_time(b) for evs in hp.gemm_events for a, b in evs) / args.steps
        two_streams = {"ms_per_step": ms_ov, "value": flops_step / ms_ov / 1e9, "unit": UNIT,
                       "gemm_ms_per_step": gemm_ms_ov, "gemm_tflops": hp.gemm_flops() / gemm_ms_ov / 1e9,
                       "what": "quantize calls on a side stream, in the shadow of the products of the groups before them"}
        del hp, h_in, h_out, hin, hout
        torch.cuda.empty_cache()
        delayed = delayed_scaling_step(cfg, host, args, flops_step)
        c2 = quantize_sweep(peaks)
        c5 = long_context_attention(peaks)
        hp = None

    if rank == 0:
        c = cfg
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp8 (e4m3/e5m2 operands, f32 accumulate)", "data": "synthetic",
            "config": {"workload": f"{c.name}: Llama-style block, tokens {c.tokens} ({c.batch}x{c.seq}), hidden "
                                   f"{c.hidden}, heads {c.n_q_heads}/{c.n_kv_heads} x {c.head_dim}, ffn {c.ffn}"
                                   f"{' gated' if c.gated else ''}; quantize + 12 GEMMs + causal attention fwd+bwd",
                       "l2": "per-step working set (GBs) exceeds the 126 MB L2; no flush needed",
                       "replicas": world, "attn_max_slack": args.attn_slack},
            "pct_of_nominal_fp8_peak": 100.0 * value / world / FP8_NOMINAL_TFLOPS,
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": e2e_steps,
                    "api": "fp8_linear_step_host x 4 + fp8_attention_step_host, then fp8_host_sync (C ABI, host buffers)",
                    "device_pointer_calls_on_three_streams": e2e_binding_value},
            "gpu_launches": acct["launches"],
            "roofline": roofline,
            "cpu_baseline": cpu_baseline,
            "attention": attention,
            "quantize": quantize,
            "two_stream_step": two_streams,
            "delayed_scaling_step": delayed,
            "c2_quantize_sweep": c2,
            "c5_long_context_attention": c5,
            "breakdown": {"gemm_ms_per_step": gemm_ms / args.steps, "gemm_tflops": gemm_tflops,
                          "gemm_tflop_per_step": acct["gemm_tflop"],
                          "attention_tflop_per_step": acct["attn_tflop"],
                          "quantize_gb_per_step": acct["quant_gb"]},
        }
        if graph_info is not None:
            line["graph"] = graph_info
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per GEMM launch, averaged over the 12 launches of one step:
# from one single-pass ncu capture of this benchmark (`--metrics dram__bytes_read.sum,dram__bytes_write.sum,
# gpu__time_duration.sum --clock-control none -k regex:gemm_fp8`), taken on the commit named in `source`.  None for
# workloads without a capture: a figure from another build says nothing about this one.
GEMM_DRAM_CAPTURE = {
    "c4": {"bytes_per_launch": 316.73e6,
           "source": "ncu, 12 launches of one c4 step, commit 2df078f: read 215.6 MB + write 101.1 MB per launch on "
                     "average, against 263 MB of operands and outputs"},
}


# ---------------------------------------------------------------------------------------------- per-kernel report
def run_report(args):
    """`--report`: every kernel of the library timed alone (CUDA events on the launching stream, 3 warm-ups, median of
    `--steps` launches).  Between launches a 256 MB buffer is written (nothing of the previous launch stays in L2) and
    then a second 256 MB buffer is read, so that the timed launch does not pay for writing the fill's dirty lines back
    (up to 126 MB: as much as a whole small kernel moves).  Prints one JSON line {"report": [...]}; the default bench
    line is not affected."""
    import numpy as np
    import torch

    import paper_2505_20524_b200 as fp8
    from paper_2505_20524_b200 import synth

    torch.cuda.set_device(0)
    fp8.binding.load()
    peaks = measured_peaks()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    scrub = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")
    rows = []

    def timed(fn):
        for _ in range(3):
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
        for i, (a, b) in enumerate(ev):
            flush.fill_(i & 0xFF)
            scrub.sum()                   # clean lines push the fill's dirty ones out before the clock starts
            a.record()
            fn()
            b.record()
        torch.cuda.synchronize()
        return float(np.median([a.elapsed_time(b) for a, b in ev]))

    def add(kernel, shape, ms, flops=None, nbytes=None):
        r = {"kernel": kernel, "shape": shape, "ms": round(ms, 4)}
        if flops is not None:
            r["tflops"] = round(flops / ms / 1e9, 1)
            r["frac_of_2x_bf16_burst"] = round(flops / ms / 1e9 / (2 * peaks["bf16_burst"]), 3)
        if nbytes is not None:
            r["gbs"] = round(nbytes / ms / 1e6, 0)
            r["frac_of_hbm"] = round(nbytes / ms / 1e6 / peaks["hbm"], 3)
        rows.append(r)

    def f32(v=0.0):
        return torch.full((1,), float(v), dtype=torch.float32, device="cuda")

    def bf16(*shape, std=1.0):
        return (std * torch.randn(shape, device="cuda")).to(torch.bfloat16)

    def codes(*shape):
        return torch.randint(0x20, 0x48, shape, dtype=torch.uint8, device="cuda")

    def cast_codes(shape, std, fmt):
        """FP8 codes of a normal tensor under just-in-time scaling: the bit activity of real operands (uniformly drawn
        codes run several per cent faster on a power-capped board)."""
        x = (std * torch.randn(shape, device="cuda")).to(torch.bfloat16)
        q = torch.empty(shape, dtype=torch.uint8, device="cuda")
        fp8.fp8_quantize(x, fmt, q, None, f32(), f32(), f32())
        return q

    # ---- quantize family (HBM): the flat sweep of workload c2 and the block tensors of c4
    for n in (1 << 24, 1 << 27, 1 << 29):
        x = bf16(n)
        q = torch.empty(n, dtype=torch.uint8, device="cuda")
        a, sc, si = f32(), f32(1.0), f32(1.0)
        add("fp8_amax", f"{n}", timed(lambda: fp8.fp8_amax(x, a)), nbytes=2 * n)
        add("fp8_cast e4m3", f"{n}", timed(lambda: fp8.fp8_cast(x, sc, fp8.E4M3, q)), nbytes=3 * n)
        add("fp8_quantize e4m3 (amax + cast)", f"{n}", timed(lambda: fp8.fp8_quantize(x, fp8.E4M3, q, None, a, sc, si)),
            nbytes=5 * n)
        del x, q
    c4 = synth.CONFIGS["c4"]
    T, H, F = c4.tokens, c4.hidden, c4.ffn
    x = bf16(T, 2 * F)
    q, qt = torch.empty((T, 2 * F), dtype=torch.uint8, device="cuda"), torch.empty((2 * F, T), dtype=torch.uint8, device="cuda")
    a, sc, si = f32(), f32(1.0), f32(1.0)
    add("fp8_quantize e5m2 + transposed copy", f"{T}x{2 * F}",
        timed(lambda: fp8.fp8_quantize(x, fp8.E5M2, q, qt, a, sc, si)), nbytes=6 * T * 2 * F)
    # the operands of the c4 QKV projection as one group: X [T,H], W [3H/2,H], dY [T,3H/2]
    gx = [bf16(T, H), bf16(3 * H // 2, H), bf16(T, 3 * H // 2)]
    gf = [fp8.E4M3, fp8.E4M3, fp8.E5M2]
    gq = [torch.empty(t.shape, dtype=torch.uint8, device="cuda") for t in gx]
    gn = sum(t.numel() for t in gx)
    gsc = torch.zeros(9, dtype=torch.float32, device="cuda")
    add("fp8_quantize_multi (X, W, dY of the QKV projection; two launches)", f"{gn}",
        timed(lambda: fp8.fp8_quantize_multi(gx, gf, gq, gsc)), nbytes=5 * gn)
    gh = [torch.zeros(1024, dtype=torch.float32, device="cuda") for _ in gx]
    ghd = [torch.zeros(1, dtype=torch.int32, device="cuda") for _ in gx]
    gs, ga, gs1, gsi1 = [f32(1.0) for _ in gx], [f32() for _ in gx], [f32() for _ in gx], [f32() for _ in gx]
    gsync = torch.zeros(6, dtype=torch.int32, device="cuda")
    add("fp8_quantize_delayed_multi (same group: codes, amax, history update, next scale; one launch)", f"{gn}",
        timed(lambda: fp8.fp8_quantize_delayed_multi(gx, gf, gq, gh, ghd, gs, ga, gs1, gsi1, 0, gsync)), nbytes=3 * gn)
    del gx, gq
    h8, h8t = torch.empty((T, F), dtype=torch.uint8, device="cuda"), torch.empty((F, T), dtype=torch.uint8, device="cuda")
    add("fp8_swiglu_cast (amax pass)", f"{T}x{F}", timed(lambda: fp8.fp8_swiglu_cast(x, None, 0, None, None, a)),
        nbytes=4 * T * F)
    add("fp8_swiglu_cast (cast + transposed copy)", f"{T}x{F}", timed(lambda: fp8.fp8_swiglu_cast(x, sc, 0, h8, h8t, None)),
        nbytes=6 * T * F)
    xa = x[:, :F].contiguous()
    par = torch.tensor([0.8, 1.3], device="cuda")
    for act, name in ((fp8.ACT_GELU, "gelu"), (fp8.ACT_XIELU, "xielu")):
        add(f"fp8_act_cast {name} (amax pass)", f"{T}x{F}", timed(lambda: fp8.fp8_act_cast(xa, act, par, None, 0, None, None, a)),
            nbytes=2 * T * F)
        add(f"fp8_act_cast {name} (cast + transposed copy)", f"{T}x{F}",
            timed(lambda: fp8.fp8_act_cast(xa, act, par, sc, 0, h8, h8t, None)), nbytes=4 * T * F)
    for act, name in ((fp8.ACT_GELU, "gelu"), (fp8.ACT_XIELU, "xielu")):
        # delayed scaling: codes and amax in one pass over the input (2 B read + 1 B written per element)
        add(f"fp8_act_cast {name} (single pass: cast + amax under a delayed scale)", f"{T}x{F}",
            timed(lambda: fp8.fp8_act_cast(xa, act, par, sc, 0, h8, None, a)), nbytes=3 * T * F)
    add("fp8_kurtosis", f"{T}x{2 * F}", timed(lambda: fp8.fp8_kurtosis(x, a)), nbytes=2 * T * 2 * F)
    kk = f32()
    add("fp8_amax_kurtosis (amax + kurtosis, one pass)", f"{T}x{2 * F}", timed(lambda: fp8.fp8_amax_kurtosis(x, a, kk)),
        nbytes=2 * T * 2 * F)
    del x, q, qt, h8, h8t, xa
    r, y, g = bf16(2 * T, H), bf16(2 * T, H, std=0.02), torch.ones(H, device="cuda")
    o_ = torch.empty_like(r)
    for mode, name in ((fp8.NORM_RMS, "rmsnorm"), (fp8.NORM_LAYERSCALE, "layerscale")):
        add(f"fp8_postnorm_residual {name}", f"{2 * T}x{H}", timed(lambda: fp8.fp8_postnorm_residual(r, y, g, mode, 1e-5, o_, a)),
            nbytes=6 * 2 * T * H)
    o8 = torch.empty((2 * T, H), dtype=torch.uint8, device="cuda")
    add("fp8_postnorm_residual_q rmsnorm (BF16 + FP8 codes + amax, delayed scale)", f"{2 * T}x{H}",
        timed(lambda: fp8.fp8_postnorm_residual_q(r, y, g, fp8.NORM_RMS, 1e-5, sc, 0, o_, o8, a)), nbytes=7 * 2 * T * H)
    del o8
    qk = bf16(2 * T, c4.n_q_heads, c4.head_dim)
    qo = torch.empty_like(qk)
    cos, sin = torch.rand((c4.seq, c4.head_dim // 2), device="cuda"), torch.rand((c4.seq, c4.head_dim // 2), device="cuda")
    for mode, name in ((fp8.QK_RMS, "rms"), (fp8.QK_TANH, "tanh"), (fp8.QK_NONE, "none")):
        add(f"fp8_qk_norm_rope {name} + rotary", f"{2 * T}x{c4.n_q_heads}x{c4.head_dim}",
            timed(lambda: fp8.fp8_qk_norm_rope(qk, mode, 0.5, 1e-6, cos, sin, c4.seq, qo, a)), nbytes=4 * qk.numel())
    q8_ = torch.empty(qk.shape, dtype=torch.uint8, device="cuda")
    add("fp8_qk_norm_rope_q rms + rotary (FP8 codes only + amax, delayed scale)", f"{2 * T}x{c4.n_q_heads}x{c4.head_dim}",
        timed(lambda: fp8.fp8_qk_norm_rope_q(qk, fp8.QK_RMS, 0.5, 1e-6, cos, sin, c4.seq, sc, 0, None, q8_, a)),
        nbytes=3 * qk.numel())
    del r, y, o_, qk, qo, q8_

    # ---- GEMMs of c3 and c4: forward / dgrad / wgrad, the producer form and the blockwise recipe
    for cname in ("c3", "c4"):
        cfg = synth.CONFIGS[cname]
        for layer, (Tt, N, K) in cfg.linear_shapes().items():
            x8, w8, dy8 = cast_codes((Tt, K), 1.0, fp8.E4M3), cast_codes((N, K), 0.02, fp8.E4M3), cast_codes((Tt, N), 1e-3, fp8.E5M2)
            x8t, w8t, dy8t = x8.t().contiguous(), w8.t().contiguous(), dy8.t().contiguous()
            s1, s2 = f32(1e-2), f32(1e-2)
            yb, dxb, dwb = (torch.empty(sh, dtype=torch.bfloat16, device="cuda") for sh in ((Tt, N), (Tt, K), (N, K)))
            fl = 2.0 * Tt * N * K
            add("fp8_linear_fwd", f"{cname} {layer} {Tt}x{N}x{K}", timed(lambda: fp8.fp8_linear_fwd(x8, w8, s1, s2, yb)), flops=fl)
            try:        # context only: the library's FP8 product on the same operands (a cuBLASLt call through torch)
                xf, wf = x8.view(torch.float8_e4m3fn), w8.view(torch.float8_e4m3fn)
                add("library FP8 GEMM, torch._scaled_mm (context)", f"{cname} {layer} {Tt}x{N}x{K}",
                    timed(lambda: torch._scaled_mm(xf, wf.t(), scale_a=s1, scale_b=s2, out_dtype=torch.bfloat16)), flops=fl)
            except Exception:
                pass
            add("fp8_linear_dgrad", f"{cname} {layer} {Tt}x{N}x{K}", timed(lambda: fp8.fp8_linear_dgrad(dy8, w8t, s1, s2, dxb)), flops=fl)
            add("fp8_linear_wgrad", f"{cname} {layer} {Tt}x{N}x{K}", timed(lambda: fp8.fp8_linear_wgrad(dy8t, x8t, s1, s2, dwb)), flops=fl)
            add("fp8_linear_dgrad_rm (W8 read in place)", f"{cname} {layer} {Tt}x{N}x{K}",
                timed(lambda: fp8.fp8_linear_dgrad_rm(dy8, w8, s1, s2, dxb)), flops=fl)
            add("fp8_linear_wgrad_rm (dY8, X8 read in place)", f"{cname} {layer} {Tt}x{N}x{K}",
                timed(lambda: fp8.fp8_linear_wgrad_rm(dy8, x8, s1, s2, dwb)), flops=fl)
            if cname == "c4":
                y8 = torch.empty((Tt, N), dtype=torch.uint8, device="cuda")
                add("fp8_linear_fwd_q (fp8 epilogue + amax)", f"{cname} {layer} {Tt}x{N}x{K}",
                    timed(lambda: fp8.fp8_linear_fwd_q(x8, w8, s1, s2, sc, fp8.E4M3, y8, a)), flops=fl)
                sx = torch.full((K // 128, Tt), 1e-2, device="cuda")
                sw = torch.full(((N + 127) // 128, K // 128), 1e-2, device="cuda")
                add("fp8_linear_fwd_blockwise", f"{cname} {layer} {Tt}x{N}x{K}",
                    timed(lambda: fp8.fp8_linear_fwd_blockwise(x8, w8, sx, sw, yb)), flops=fl)
                if N % 128 == 0:
                    sdy = torch.full((N // 128, Tt), 1e-2, device="cuda")
                    add("fp8_linear_dgrad_blockwise (W8 and its block scales read in place)", f"{cname} {layer} {Tt}x{N}x{K}",
                        timed(lambda: fp8.fp8_linear_dgrad_blockwise(dy8, w8, sdy, sw, dxb)), flops=fl)
                    del sdy
                sdt = torch.full(((Tt + 127) // 128, N), 1e-2, device="cuda")
                sxt = torch.full(((Tt + 127) // 128, K), 1e-2, device="cuda")
                add("fp8_linear_wgrad_blockwise (128x1 blocks, operands read in place)", f"{cname} {layer} {Tt}x{N}x{K}",
                    timed(lambda: fp8.fp8_linear_wgrad_blockwise(dy8, x8, sdt, sxt, dwb)), flops=fl)
                xb = bf16(Tt, K)
                add("fp8_quantize_blockwise 1x128", f"{Tt}x{K}", timed(lambda: fp8.fp8_quantize_blockwise(xb, 1, 0, x8, sx)),
                    nbytes=3 * Tt * K)
                add("fp8_quantize_blockwise 128x1", f"{Tt}x{K}",
                    timed(lambda: fp8.fp8_quantize_blockwise(xb, fp8.FP8_BLOCK_128x1, 0, x8, sxt)), nbytes=3 * Tt * K)
                del xb, y8, sx, sw, sdt, sxt
            del x8, w8, dy8, x8t, w8t, dy8t, yb, dxb, dwb

    # ---- grouped (mixture-of-experts) forward product: 8 experts, 2 active, c3-sized FFN
    c3 = synth.CONFIGS["c3"]
    E, Tr = 8, 2 * c3.tokens                                   # every token is routed to 2 experts
    rng = np.random.default_rng(1)
    wts = np.maximum(1e-3, 1 + 0.3 * rng.standard_normal(E))
    sizes = np.floor(wts / wts.sum() * Tr).astype(int)
    sizes[-1] += Tr - sizes.sum()
    offs = torch.from_numpy(np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)).cuda()
    Ng, Kg = 2 * c3.ffn, c3.hidden
    x8, w8 = codes(Tr, Kg), codes(E, Ng, Kg)
    yb = torch.empty((Tr, Ng), dtype=torch.bfloat16, device="cuda")
    s1, swg = f32(1e-2), torch.full((E,), 1e-2, device="cuda")
    add("fp8_grouped_linear_fwd (8 experts, uneven)", f"{Tr} rows x {Ng} x {Kg}",
        timed(lambda: fp8.fp8_grouped_linear_fwd(x8, w8, s1, swg, offs, yb)), flops=2.0 * Tr * Ng * Kg)
    dy8 = codes(Tr, Ng)
    dxb = torch.empty((Tr, Kg), dtype=torch.bfloat16, device="cuda")
    add("fp8_grouped_linear_dgrad (8 experts, uneven, weights in place)", f"{Tr} rows x {Ng} x {Kg}",
        timed(lambda: fp8.fp8_grouped_linear_dgrad(dy8, w8, s1, swg, offs, dxb)), flops=2.0 * Tr * Ng * Kg)
    dwb = torch.empty((E, Ng, Kg), dtype=torch.bfloat16, device="cuda")
    offs_host = [int(v) for v in offs.cpu().tolist()]
    add("fp8_grouped_linear_wgrad (8 experts, uneven, one launch per expert)", f"{Tr} rows x {Ng} x {Kg}",
        timed(lambda: fp8.fp8_grouped_linear_wgrad(dy8, x8, s1, s1, offs_host, dwb)), flops=2.0 * Tr * Ng * Kg)
    wsg = torch.empty(fp8.fp8_grouped_linear_wgrad_workspace_bytes(E, Ng), dtype=torch.uint8, device="cuda")
    add("fp8_grouped_linear_wgrad_dev (8 experts, uneven, one launch, device offsets)", f"{Tr} rows x {Ng} x {Kg}",
        timed(lambda: fp8.fp8_grouped_linear_wgrad_dev(dy8, x8, s1, s1, offs, dwb, wsg)), flops=2.0 * Tr * Ng * Kg)
    del x8, w8, yb, dy8, dxb, dwb, wsg

    # ---- attention of c3, c4, c5 (causal)
    for cname in ("c3", "c4", "c5"):
        cfg = synth.CONFIGS[cname]
        B, N, Hq, Hkv, d = cfg.batch, cfg.seq, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        sgn = torch.randint(0, 2, (B, N, Hq, d), dtype=torch.uint8, device="cuda") << 7
        q8 = codes(B, N, Hq, d) | sgn
        k8 = codes(B, N, Hkv, d) | (torch.randint(0, 2, (B, N, Hkv, d), dtype=torch.uint8, device="cuda") << 7)
        v8 = codes(B, N, Hkv, d)
        do8 = torch.randint(0x20, 0x40, (B, N, Hq, d), dtype=torch.uint8, device="cuda") | sgn
        O = torch.empty((B, N, Hq, d), dtype=torch.bfloat16, device="cuda")
        LSE = torch.empty((B, Hq, N), dtype=torch.float32, device="cuda")
        dq, dk, dv = torch.empty_like(O), torch.empty((B, N, Hkv, d), dtype=torch.bfloat16, device="cuda"), None
        dv = torch.empty_like(dk)
        ws = torch.empty(fp8.fp8_attention_workspace_bytes(1, B, N, Hq, Hkv, d), dtype=torch.uint8, device="cuda")
        s1, dss, s = f32(0.05), f32(64.0), d ** -0.5
        fl = 2.0 * B * Hq * N * N * d
        shape = f"{cname} B{B} N{N} H{Hq}/{Hkv} d{d}"
        add("fp8_attention_fwd", shape, timed(lambda: fp8.fp8_attention_fwd(q8, k8, v8, s1, s1, s1, s, True, O, LSE, None)), flops=fl)
        add("fp8_attention_fwd (reference maximum with slack 2^2, c_P = 112)", shape,
            timed(lambda: fp8.fp8_attention_fwd(q8, k8, v8, s1, s1, s1, s, True, O, LSE, None, p_scale=112.0,
                                                max_slack=2.0)), flops=fl)
        add("fp8_attention_bwd", shape,
            timed(lambda: fp8.fp8_attention_bwd(q8, k8, v8, do8, O, LSE, s1, s1, s1, s1, s, dss, True, dq, dk, dv, ws)),
            flops=2.5 * fl)
        del q8, k8, v8, do8, O, LSE, dq, dk, dv, ws
    status = fp8.fp8_device_status()
    print(json.dumps({"report": rows, "device_status": status, "steps": args.steps,
                      "peaks": {"hbm_gbs": peaks["hbm"], "bf16_tflops_burst": peaks["bf16_burst"], "source": peaks["source"]}}),
          flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c4", choices=["c1", "c3", "c4", "c5"])
    ap.add_argument("--report", action="store_true", help="time every kernel of the library alone and print a table")
    ap.add_argument("--attn-slack", type=float, default=0.0,
                    help="tau of the attention forward's reference maximum (default 0 = exact running maximum; the "
                         "contract line is quoted with 0)")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the two extra workloads of the default line (c2 quantize sweep, c5 attention)")
    ap.add_argument("--graph", action="store_true",
                    help="also time the step replayed from a CUDA graph (extra key \"graph\"; the contract keys stay eager)")
    args = ap.parse_args()
    if args.report:
        return run_report(args)
    from paper_2505_20524_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
