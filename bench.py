#!/usr/bin/env python
"""Benchmark of the fused RoPE + causal attention path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--extras 0|1]

Prints ONE JSON line.  A step is one fused forward pass (rotate Q and K on chip, QK^T, causal
mask, online softmax, PV, O and L written) over the Llama-3-8B attention shape (B=1, Hq=32,
Hkv=8, S=4096, D=128, bf16); `value` is algorithmic TFLOP/s (two contractions over the kept
(query, key) pairs only).  The cos/sin table is set-up, built once before the timed region.

Inputs are seeded synthetic N(0,1) tensors of that shape, resident in HBM; the timed steps rotate
over several independent input sets whose total size exceeds L2, so no step finds its inputs
cached.  `e2e` measures the same step through the host-buffer entry point (pinned host memory,
copies inside the timed region).  `--impl reference` times the fp64 CPU oracle on the host cores.
With N > 1 (torchrun) every rank runs the same per-GPU workload (the path shards over independent
(batch, kv-head) units with no exchange step); times are the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2609_13612_b200 import shard, synth  # noqa: E402

METRIC = "fused RoPE+causal attention TFLOP/s (bf16 fwd/bwd) and % of B200 tensor peak"
UNIT = "TFLOP/s"
L2_BYTES = 126 * 1024 * 1024
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture), by kernel and workload.
# A kernel or workload that has no entry reports "traffic": null instead of a figure that belongs to another one.
KERNEL_TRAFFIC_BYTES = {
    ("attn_fwd_kernel<128,2,rope>", "c2_llama3_8b_fwd"): 55.2e6,
}
RIDGE_CONTEXT = {"paper_ampere_flop_per_byte": 152, "paper_hopper_flop_per_byte": 300}
PAPER_CONTEXT = {
    "rtx3090_fused_vs_flex_prerotate_rope_causal": "2.10x (RTX 3090, fp16, B=4 H=12 D=64, N=4096)",
    "h100_llama3_8b_training_step_vs_sdpa": "within ~5% (H100 NVL, fp16, N=2048: 7.65 ms vs 7.27 ms)",
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d["bf16_tflops_sustained"]),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4,
                 "hw_power_brake_slowdown": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.0002)

    def mark(self):
        """Number of samples taken so far (to tell the samples of the timed region from later ones)."""
        return len(self.samples)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_rate(w: synth.Workload, budget_s: float):
    """Time the oracle (as it stands) on a row sample of workload w sized for about budget_s."""
    import oracle
    t = synth.draw_all(w)
    pilot_rows = list(range(w.S - 1, -1, -max(1, w.S // 64)))
    t0 = time.perf_counter()
    oracle.run_workload(w, t, rows=pilot_rows)
    dt = max(time.perf_counter() - t0, 1e-6)
    pairs = lambda rows: float(sum(min(i + 1, (w.window + 1) if w.window >= 0 else i + 1) for i in rows))
    rate = pairs(pilot_rows) / dt
    total = float(w.kept_pairs_per_head())
    stride = max(1, int(math.ceil(total / (rate * budget_s))))
    rows = list(range(w.S - 1, -1, -stride))
    t0 = time.perf_counter()
    oracle.run_workload(w, t, rows=rows)
    dt = time.perf_counter() - t0
    flops = 4.0 * w.D * pairs(rows) * w.B * w.Hq
    return flops / dt / 1e12, "every %d-th query row of every head (%d rows, %.1f s)" % (stride, len(rows), dt), dt


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    per_step = max(1.0, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    vals, secs, sample = [], [], ""
    for i in range(args.warmup + args.steps):
        v, sample, dt = oracle_rate(w, per_step)
        if i >= args.warmup:
            vals.append(v)
            secs.append(dt)
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": float(np.mean(secs)) * 1e3,   # one step = one bounded sample of the workload (see cpu_baseline.sample)
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "S": w.S, "D": w.D,
                                        "variant": "rope(theta=%g)+causal" % w.theta},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--extras", type=int, default=1, help="also time configs 3-5, the separate-RoPE arm and the sweep")
    ap.add_argument("--cpu-baseline", type=int, default=1)
    ap.add_argument("--profile", default="", choices=["", "fwd", "hybrid", "bwd", "bwd2", "rope", "decode", "fwd_c3", "fwd_d64", "bwd_d64", "blocks", "fp8"],
                    help="run only a few launches of one path (for ncu captures) and exit")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    w = synth.CONFIGS[1]

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import paper_2609_13612_b200 as af
    from paper_2609_13612_b200 import binding

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peaks = measured_peaks()

    def to_dev(x):
        return torch.from_numpy(synth.bf16_bits(x).view(np.int16)).view(torch.bfloat16).to(dev)

    def make_sets(wl, n_sets):
        base = {k: to_dev(v) for k, v in synth.draw_all(wl).items()}
        sets = [base]
        for s in range(1, n_sets):
            sets.append({k: torch.roll(v, shifts=s, dims=1).contiguous() for k, v in base.items()})
        return sets

    def specs(wl):
        rope = af.RopeSpec(theta=wl.theta, rotary_dim=wl.R, pos_offset=wl.pos_offset)
        sl = wl.alibi_slopes()
        mask = af.MaskSpec(causal=wl.causal, window=wl.window,
                           alibi_slopes=torch.from_numpy(sl).to(dev) if sl is not None else None)
        return rope, mask, af.rope_table(rope, wl.S, device=dev)

    def input_bytes(wl):
        return 2 * wl.B * wl.S * wl.D * (wl.Hq + 2 * wl.Hkv)

    def n_sets_for(wl):
        return max(2, int(math.ceil(2.0 * L2_BYTES / input_bytes(wl))) + 1) if input_bytes(wl) < 2 * L2_BYTES else 1

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        """K steps between barrier+sync, plus per-launch CUDA-event durations on the launching stream."""
        for i in range(warmup):
            fn(i)
        barrier()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        t0 = time.perf_counter()
        start = torch.cuda.Event(enable_timing=True)
        stop = torch.cuda.Event(enable_timing=True)
        start.record()
        for i in range(steps):
            evs[i][0].record()
            fn(i)
            evs[i][1].record()
        stop.record()
        barrier()
        wall_ms = (time.perf_counter() - t0) * 1e3
        total_ms = start.elapsed_time(stop)
        per = [a.elapsed_time(b) for a, b in evs]
        if dist is not None:
            tt = torch.tensor([total_ms], device=dev, dtype=torch.float64)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            total_ms = float(tt.item())
        return total_ms, per, wall_ms

    if args.profile == "decode":
        # Flash Decoding on the Llama-3-70B geometry of the paper's decode table (64 q / 8 kv heads, 32768 keys)
        gq = torch.Generator(device=dev).manual_seed(7)
        qd = torch.randn(1, 64, 128, device=dev, generator=gq).to(torch.bfloat16)
        kc = [torch.randn(1, 8, 32768, 128, device=dev, generator=gq).to(torch.bfloat16) for _ in range(3)]
        vc = [torch.randn(1, 8, 32768, 128, device=dev, generator=gq).to(torch.bfloat16) for _ in range(3)]
        for i in range(6):
            af.decode(qd, kc[i % 3], vc[i % 3], af.MaskSpec(True, -1, None), 128 ** -0.5)
        torch.cuda.synchronize()
        print(json.dumps({"profile": "decode", "workload": "llama3_70b_decode_32768", "device_status": af.device_status()[0]}))
        return
    if args.profile == "fp8":
        # the opt-in forward with E4M3 operands on the Llama-3-8B shape (causal, no rotation inside)
        wl = synth.CONFIGS[1]
        g8 = torch.Generator(device=dev).manual_seed(11)
        x8 = {}
        for name, H_ in (("q", wl.Hq), ("k", wl.Hkv), ("v", wl.Hkv)):
            x = torch.randn((wl.B, H_, wl.S, wl.D), device=dev, generator=g8)
            sc = float(x.abs().max()) / 448.0
            y = (x / sc).to(torch.float8_e4m3fn)
            x8[name] = (y.transpose(2, 3).contiguous() if name == "v" else y, sc)
        for _ in range(3):
            af.fwd_fp8(x8["q"][0], x8["k"][0], x8["v"][0], af.MaskSpec(causal=True), wl.scale, x8["q"][1], x8["k"][1], x8["v"][1])
        torch.cuda.synchronize()
        print(json.dumps({"profile": "fp8", "workload": wl.name + " (E4M3 operands, no RoPE)", "device_status": af.device_status()[0]}))
        return
    if args.profile:
        # a handful of launches of one path on its configuration, nothing else: the target of ncu captures
        wl = {"fwd": synth.CONFIGS[1], "hybrid": synth.CONFIGS[1], "bwd": synth.CONFIGS[4], "bwd2": synth.CONFIGS[4],
              "rope": synth.CONFIGS[3], "fwd_c3": synth.CONFIGS[2],
              "fwd_d64": synth.Workload("gpt2_small_geometry_d64", 4, 12, 12, 4096, 64, theta=1.0e4, seed_id=51),
              "bwd_d64": synth.Workload("gpt2_small_geometry_d64", 4, 12, 12, 4096, 64, theta=1.0e4, backward=True, seed_id=51),
              "blocks": synth.Workload("bigbird_d64_n4096", 4, 12, 12, 4096, 64, theta=1.0e4, causal=False, seed_id=53)}[args.profile]
        r, m, tb = specs(wl)
        t = {k: to_dev(v) for k, v in synth.draw_all(wl).items()}
        if args.profile == "blocks":   # the BigBird-like mask of the block-sparse extra (12 % of the 32 x 32 blocks)
            rng_ = np.random.Generator(np.random.PCG64(np.random.SeedSequence([20260913, 901])))
            act = np.eye(32, dtype=bool)
            act[:, 0] = True
            act[0, :] = True
            act[np.arange(32), rng_.integers(0, 32, size=32)] = True
            bmask = af.BlockMask(act, device=dev)
        for _ in range(3):
            if args.profile == "rope":
                af.rope(t["q"], r, tb)
            elif args.profile == "hybrid":
                af.fwd_hybrid(t["q"], t["k"], t["v"], r, tb, m, wl.scale)
            elif args.profile == "blocks":
                af.fwd_blocks(t["q"], t["k"], t["v"], r, tb, m, wl.scale, bmask)
            else:
                o_, l_ = af.fwd(t["q"], t["k"], t["v"], r, tb, m, wl.scale)
                if args.profile in ("bwd", "bwd2", "bwd_d64"):   # the sequence the library picks (one-pass here); bwd2: two kernels
                    with af.option(af.OPT_BWD_ONEPASS, 0 if args.profile == "bwd2" else 1):
                        af.bwd(t["q"], t["k"], t["v"], o_, l_, t["do"], r, tb, m, wl.scale)
        torch.cuda.synchronize()
        print(json.dumps({"profile": args.profile, "workload": wl.name, "device_status": af.device_status()[0]}))
        return

    # ------------------------------------------------------------------ headline: fused forward, config 2
    rope, mask, table = specs(w)
    sets = make_sets(w, n_sets_for(w))
    o = torch.empty((w.B, w.Hq, w.S, w.D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((w.B, w.Hq, w.S), dtype=torch.float32, device=dev)

    def step(i):
        s = sets[i % len(sets)]
        af.fwd(s["q"], s["k"], s["v"], rope, table, mask, w.scale, out=o, lse=lse)

    with ClockSampler(local) as clk:
        total_ms, per, _ = timed(step, args.steps, args.warmup)
        n_timed = clk.mark()
        # A short run (the timed region of 20 steps lasts a few milliseconds) yields only a few NVML samples: the
        # same step keeps running, untimed, until the sampler has seen the clocks under this load for at least 30 ms.
        t_end = time.perf_counter() + 0.03
        i_extra = 0
        while time.perf_counter() < t_end or clk.mark() < 12:
            step(i_extra)
            i_extra += 1
            if i_extra % 8 == 0:
                torch.cuda.synchronize()
            if i_extra > 20000:
                break
        torch.cuda.synchronize()
    code, detail = af.device_status()
    if code != 0:
        raise SystemExit("device-side wait ran out (0x%x): numbers invalid" % detail)
    ms_per_step = total_ms / args.steps
    flops = w.fwd_flops()
    # whole-job throughput: what all ranks processed (every rank runs the same per-GPU workload) over the slowest
    # rank's time (total_ms is already the max over ranks)
    value = shard.aggregate_throughput([flops] * world, ms_per_step * 1e-3) / 1e12
    kern_ms = float(np.mean(per))
    achieved = flops / (kern_ms * 1e-3) / 1e12
    roofline = {"bound": "tensor", "kernel": "attn_fwd_kernel<128,2,rope>", "achieved": achieved,
                "peak": peaks["bf16_tflops"], "peak_kind": "burst bf16 dense, %s" % peaks["source"], "unit": UNIT,
                "frac": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0,
                "traffic": KERNEL_TRAFFIC_BYTES.get(("attn_fwd_kernel<128,2,rope>", w.name)), "kernel_ms": kern_ms,
                "algorithmic_flops_per_launch": flops}

    # ------------------------------------------------------------------ e2e: host buffers through the C-ABI
    hq, hk, hv = (sets[0][k].cpu().pin_memory() for k in ("q", "k", "v"))
    ho = torch.empty_like(hq).pin_memory()
    hl = torch.empty((w.B, w.Hq, w.S), dtype=torch.float32).pin_memory()
    staging = torch.empty(binding.fwd_host_staging_bytes(w.B, w.Hq, w.Hkv, w.S, w.D), dtype=torch.uint8, device=dev)

    def step_host(i):
        af.fwd_host(hq, hk, hv, rope, table, mask, w.scale, ho, hl, staging)

    e2e_steps = max(3, min(args.steps, 50))
    e2e_ms, _, _ = timed(step_host, e2e_steps, 3)
    e2e_val = shard.aggregate_throughput([flops] * world, e2e_ms / e2e_steps * 1e-3) / 1e12
    h2d = int(hq.numel() * 2 + hk.numel() * 2 + hv.numel() * 2)
    d2h = int(ho.numel() * 2 + hl.numel() * 4)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "Hq": w.Hq, "Hkv": w.Hkv, "S": w.S, "D": w.D,
                   "variant": "rope(theta=%g, all dims)+causal, scale 1/sqrt(D), forward" % w.theta,
                   "l2": "inputs rotate over %d independent sets (%.0f MB total > 126 MB L2)" % (
                       len(sets), len(sets) * input_bytes(w) / 1e6),
                   "sharding": "replicated per-GPU workload, no collective" if world > 1 else "single GPU"},
        "clocks": dict(clk.summary(), samples_in_timed_region=n_timed,
                       note="sampled over warm-up, timed region and the same step continued untimed for 30 ms"),
        "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": args.steps,
        "roofline": roofline,
        "pct_of_tensor_peak": {"measured_burst_%.0f" % peaks["bf16_tflops"]: 100 * value / world / peaks["bf16_tflops"],
                               "measured_sustained_%.0f" % peaks["bf16_tflops_sustained"]:
                                   100 * value / world / peaks["bf16_tflops_sustained"],
                               "nominal_2250": 100 * value / world / 2250.0},
        "paper_context": PAPER_CONTEXT,
    }

    # ------------------------------------------------------------------ extras (rank 0's GPU only, short runs)
    if args.extras and rank == 0:
        ex = {}
        k_ex, w_ex = 20, 5

        def fwd_ms(wl, fused=True, sets_=None, hybrid=False):
            r, m, tb = specs(wl)
            ss = sets_ or make_sets(wl, n_sets_for(wl))
            oo = torch.empty((wl.B, wl.Hq, wl.S, wl.D), dtype=torch.bfloat16, device=dev)
            ll = torch.empty((wl.B, wl.Hq, wl.S), dtype=torch.float32, device=dev)
            norope = af.RopeSpec()
            if hybrid:
                # third arm: K rotated once by the RoPE pass (into a workspace), Q rotated inside the kernel
                wsk = torch.empty(ss[0]["k"].numel() * 2, dtype=torch.uint8, device=dev)
                f = lambda i: af.fwd_hybrid(ss[i % len(ss)]["q"], ss[i % len(ss)]["k"], ss[i % len(ss)]["v"], r, tb, m,
                                            wl.scale, out=oo, lse=ll, workspace=wsk)
            elif fused:
                f = lambda i: af.fwd(ss[i % len(ss)]["q"], ss[i % len(ss)]["k"], ss[i % len(ss)]["v"], r, tb, m,
                                     wl.scale, out=oo, lse=ll)
            else:
                qr = torch.empty_like(ss[0]["q"])
                kr = torch.empty_like(ss[0]["k"])

                def f(i):
                    s = ss[i % len(ss)]
                    af.rope(s["q"], r, tb, out=qr)
                    af.rope(s["k"], r, tb, out=kr)
                    af.fwd(qr, kr, s["v"], norope, None, m, wl.scale, out=oo, lse=ll)
            t, _, _ = timed(f, k_ex, w_ex)
            return t / k_ex, ss

        # Optional forward mode: key tiles rotated in packed bf16 arithmetic from TMA-fed tiles of the table's bf16
        # copy (a tuning option of the library).  Faster, about 1.4 times the rounding error on rotated keys;
        # forward only, off by default - the headline above is the default fp32 rotation.
        wl = synth.CONFIGS[1]
        ms_d, ss = fwd_ms(wl, True)
        with af.option(af.OPT_FWD_KEYS_BF16, 1):
            ms_b, _ = fwd_ms(wl, True, ss)
        ex["c2_keys_rotated_in_packed_bf16"] = {"default_fwd_ms": ms_d, "default_fwd_tflops": wl.fwd_flops() / ms_d / 1e9,
                                                "mode_fwd_ms": ms_b, "mode_fwd_tflops": wl.fwd_flops() / ms_b / 1e9,
                                                "mode_frac_of_measured_burst_peak": wl.fwd_flops() / ms_b / 1e9 / peaks["bf16_tflops"]}
        del ss
        torch.cuda.empty_cache()
        # Opt-in forward with 8-bit E4M3 operands (no rotation inside; its own stated tolerance, never part of the bf16
        # figures): the Llama-3-8B shape, causal, inputs quantised here with per-tensor scales, 8 input sets (> L2).
        n8 = 8
        sets8 = []
        for i in range(n8):
            qkv = {}
            for name, H_ in (("q", wl.Hq), ("k", wl.Hkv), ("v", wl.Hkv)):
                x = torch.randn((wl.B, H_, wl.S, wl.D), device=dev, generator=torch.Generator(device=dev).manual_seed(100 + 3 * i + len(name) + ord(name[0])))
                sc = float(x.abs().max()) / 448.0
                x8 = (x / sc).to(torch.float8_e4m3fn)
                qkv[name] = (x8.transpose(2, 3).contiguous() if name == "v" else x8, sc)
            sets8.append(qkv)
        m8 = af.MaskSpec(causal=True)
        t8, _, _ = timed(lambda i: af.fwd_fp8(sets8[i % n8]["q"][0], sets8[i % n8]["k"][0], sets8[i % n8]["v"][0], m8, wl.scale,
                                              sets8[i % n8]["q"][1], sets8[i % n8]["k"][1], sets8[i % n8]["v"][1]), k_ex, w_ex)
        ex["c2_shape_fp8_e4m3_operands_no_rope"] = {
            "fwd_ms": t8 / k_ex, "fwd_tflops": wl.fwd_flops() / (t8 / k_ex) / 1e9,
            "note": "opt-in; probabilities rounded to E4M3, stated bound max abs 1e-1 / mean abs 8e-3 against the oracle on the "
                    "dequantised inputs; compare with the bf16 kernel without RoPE on the same shape (rotation_calculus_sweep, S = 4096)"}
        del sets8
        torch.cuda.empty_cache()
        # Composed variants of Section 3.1 on the same shape: a shared additive bias [1, 1, S, S] (fp32, 64 MB, read once per
        # head: the variant is bound by that traffic) and the ReLU normaliser, forward and backward.
        sv_ = make_sets(synth.Workload("variants_on_c2_shape", wl.B, wl.Hq, wl.Hkv, wl.S, wl.D, theta=wl.theta, backward=True,
                                       seed_id=55), 1)[0]
        rv, mv, tv_ = specs(wl)
        bias_v = torch.randn((1, 1, wl.S, wl.S), device=dev, generator=torch.Generator(device=dev).manual_seed(5)) * 0.5
        wsv = torch.empty(af.bwd_workspace_bytes(wl.B, wl.Hq, wl.Hkv, wl.S, wl.D, onepass=False), dtype=torch.uint8, device=dev)
        var = {}
        for tag, kw in (("additive_bias", dict(bias=bias_v)), ("relu_attention", dict(normaliser="relu"))):
            tf_, _, _ = timed(lambda i: af.fwd_variant(sv_["q"], sv_["k"], sv_["v"], rv, tv_, mv, wl.scale, **kw), k_ex, w_ex)
            ov, lv = af.fwd_variant(sv_["q"], sv_["k"], sv_["v"], rv, tv_, mv, wl.scale, **kw)
            tb_, _, _ = timed(lambda i: af.bwd_variant(sv_["q"], sv_["k"], sv_["v"], ov, lv, sv_["do"], rv, tv_, mv, wl.scale,
                                                       workspace=wsv, **kw), k_ex, w_ex)
            var[tag] = {"fwd_ms": tf_ / k_ex, "fwd_tflops": wl.fwd_flops() / (tf_ / k_ex) / 1e9,
                        "bwd_ms": tb_ / k_ex, "bwd_tflops": 2.5 * wl.fwd_flops() / (tb_ / k_ex) / 1e9}
        ex["composed_variants_on_c2_shape"] = var
        del sv_, bias_v, wsv
        torch.cuda.empty_cache()
        for wl in synth.CONFIGS[1:4]:
            ms_f, ss = fwd_ms(wl, True)
            ms_s, _ = fwd_ms(wl, False, ss)
            ms_h, _ = fwd_ms(wl, True, ss, hybrid=True)
            ex[wl.name] = {"fused_fwd_ms": ms_f, "fused_fwd_tflops": wl.fwd_flops() / ms_f / 1e9,
                           "separate_rope_fwd_ms": ms_s, "separate_rope_fwd_tflops": wl.fwd_flops() / ms_s / 1e9,
                           "fused_over_separate_speedup": ms_s / ms_f,
                           "hybrid_fwd_ms": ms_h, "hybrid_fwd_tflops": wl.fwd_flops() / ms_h / 1e9,
                           "hybrid_frac_of_measured_burst_peak": wl.fwd_flops() / ms_h / 1e9 / peaks["bf16_tflops"]}
            del ss
            torch.cuda.empty_cache()
        # config 5: forward + backward
        w5 = synth.CONFIGS[4]
        r5, m5, t5 = specs(w5)
        s5 = make_sets(w5, n_sets_for(w5))
        o5, l5 = af.fwd(s5[0]["q"], s5[0]["k"], s5[0]["v"], r5, t5, m5, w5.scale)
        ws = torch.empty(af.bwd_workspace_bytes(w5.B, w5.Hq, w5.Hkv, w5.S, w5.D), dtype=torch.uint8, device=dev)

        def fb(i):
            s = s5[i % len(s5)]
            af.fwd(s["q"], s["k"], s["v"], r5, t5, m5, w5.scale, out=o5, lse=l5)
            af.bwd(s["q"], s["k"], s["v"], o5, l5, s["do"], r5, t5, m5, w5.scale, workspace=ws)

        def bonly(i):
            s = s5[i % len(s5)]
            af.bwd(s["q"], s["k"], s["v"], o5, l5, s["do"], r5, t5, m5, w5.scale, workspace=ws)

        wsk5 = torch.empty(s5[0]["k"].numel() * 2, dtype=torch.uint8, device=dev)

        def fb_hybrid(i):   # the same step with the hybrid forward (K rotated once by the RoPE pass)
            s = s5[i % len(s5)]
            af.fwd_hybrid(s["q"], s["k"], s["v"], r5, t5, m5, w5.scale, out=o5, lse=l5, workspace=wsk5)
            af.bwd(s["q"], s["k"], s["v"], o5, l5, s["do"], r5, t5, m5, w5.scale, workspace=ws)

        t_fb, _, _ = timed(fb, k_ex, w_ex)
        t_fbh, _, _ = timed(fb_hybrid, k_ex, w_ex)
        t_b, _, _ = timed(bonly, k_ex, w_ex)
        with af.option(af.OPT_BWD_ONEPASS, 0):   # the two-kernel sequence (bit-reproducible dQ) on the same inputs
            t_b2, _, _ = timed(bonly, k_ex, w_ex)
        ex[w5.name] = {"fwd_bwd_ms": t_fb / k_ex,
                       "fwd_bwd_tflops": (w5.fwd_flops() + w5.bwd_flops()) / (t_fb / k_ex) / 1e9,
                       "hybrid_fwd_bwd_ms": t_fbh / k_ex,
                       "hybrid_fwd_bwd_tflops": (w5.fwd_flops() + w5.bwd_flops()) / (t_fbh / k_ex) / 1e9,
                       "bwd_ms": t_b / k_ex, "bwd_tflops": w5.bwd_flops() / (t_b / k_ex) / 1e9,
                       "bwd_pct_of_measured_peak": 100 * w5.bwd_flops() / (t_b / k_ex) / 1e9 / peaks["bf16_tflops"],
                       "bwd_sequence": "one-pass (dK, dV and dQ shares from one kernel per key tile)",
                       "bwd_two_kernel_sequence_ms": t_b2 / k_ex,
                       "bwd_two_kernel_sequence_tflops": w5.bwd_flops() / (t_b2 / k_ex) / 1e9}
        del s5
        torch.cuda.empty_cache()

        def bwd_ms(wl):
            r, m, tb = specs(wl)
            ss = make_sets(wl, min(2, n_sets_for(wl)))
            o_, l_ = af.fwd(ss[0]["q"], ss[0]["k"], ss[0]["v"], r, tb, m, wl.scale)
            wsb = torch.empty(af.bwd_workspace_bytes(wl.B, wl.Hq, wl.Hkv, wl.S, wl.D), dtype=torch.uint8, device=dev)
            t, _, _ = timed(lambda i: af.bwd(ss[i % len(ss)]["q"], ss[i % len(ss)]["k"], ss[i % len(ss)]["v"], o_, l_,
                                             ss[i % len(ss)]["do"], r, tb, m, wl.scale, workspace=wsb), k_ex, w_ex)
            return t / k_ex

        # the single-GPU geometry of the paper's tables (Section 5: B = 4, 12 heads, D = 64, N = 4096), RoPE + causal
        wg = synth.Workload("gpt2_small_geometry_d64", 4, 12, 12, 4096, 64, theta=1.0e4, backward=True, seed_id=51)
        ms_f, ss = fwd_ms(wg, True)
        ms_s, _ = fwd_ms(wg, False, ss)
        del ss
        torch.cuda.empty_cache()
        ms_b = bwd_ms(wg)
        ex[wg.name] = {"fused_fwd_ms": ms_f, "fused_fwd_tflops": wg.fwd_flops() / ms_f / 1e9,
                       "separate_rope_fwd_ms": ms_s, "fused_over_separate_speedup": ms_s / ms_f,
                       "bwd_ms": ms_b, "bwd_tflops": wg.bwd_flops() / ms_b / 1e9}
        # the composed variant (window + ALiBi) through the backward, on config 3's shape
        c3 = synth.CONFIGS[2]
        wc = synth.Workload("c3_composed_backward", c3.B, c3.Hq, c3.Hkv, c3.S, c3.D, theta=c3.theta, window=c3.window,
                            alibi=True, backward=True, seed_id=52)
        ms_b = bwd_ms(wc)
        ex[wc.name] = {"bwd_ms": ms_b, "bwd_tflops": wc.bwd_flops() / ms_b / 1e9}
        torch.cuda.empty_cache()
        # Flash Decoding (Section 4.2, the paper's decode table): query length 1, D = 128, B = 1.  HBM-bound: the
        # algorithmic bytes are the K and V caches, read once.  Caches rotate over sets larger than L2 in total.
        # Timed twice: as a replayed CUDA graph (device time per call) and through the C-ABI call from the host.
        dec = []
        for name, Hq_, Hkv_, N_, paper_ms in (("llama3_8b", 32, 8, 4096, 0.034), ("llama3_70b", 64, 8, 32768, 0.184),
                                              ("mistral_7b", 32, 8, 16384, 0.072)):
            nbytes = 2 * Hkv_ * N_ * 128 * 2
            nsets = max(2, int(300e6 // nbytes) + 1)
            gq = torch.Generator(device=dev).manual_seed(7)
            qd = torch.randn(1, Hq_, 128, device=dev, generator=gq).to(torch.bfloat16)
            kcs = [torch.randn(1, Hkv_, N_, 128, device=dev, generator=gq).to(torch.bfloat16) for _ in range(nsets)]
            vcs = [torch.randn(1, Hkv_, N_, 128, device=dev, generator=gq).to(torch.bfloat16) for _ in range(nsets)]
            md = af.MaskSpec(True, -1, None)
            od = torch.empty(1, Hq_, 128, device=dev, dtype=torch.bfloat16)
            ld = torch.empty(1, Hq_, device=dev, dtype=torch.float32)
            shp = binding._Shape(1, Hq_, Hkv_, N_, 128)
            nsp = af.lib().attnfuse_decode_splits(__import__("ctypes").byref(shp))
            wsd = af.decode_workspace(1, Hq_, Hkv_, N_, 128, nsp, device=dev)
            call = lambda i: af.decode(qd, kcs[i % nsets], vcs[i % nsets], md, 128 ** -0.5, n_splits=nsp, out=od, lse=ld,
                                       workspace=wsd)
            t_host, _, _ = timed(call, 2 * k_ex, w_ex)
            side = torch.cuda.Stream(device=dev)
            gr = torch.cuda.CUDAGraph()
            with torch.cuda.stream(side):
                with torch.cuda.graph(gr, stream=side):
                    for i in range(nsets):
                        call(i)
            t_gr, _, _ = timed(lambda i: gr.replay(), k_ex, w_ex)
            us = t_gr / k_ex / nsets * 1e3
            dec.append({"geometry": name, "Hq": Hq_, "Hkv": Hkv_, "cache": N_, "n_splits": nsp, "kv_bytes": nbytes,
                        "graph_replay_us": us, "GB/s": nbytes / us / 1e3, "frac_of_measured_hbm": nbytes / us / 1e3 / peaks["hbm_gbs"],
                        "c_abi_call_from_host_us": t_host / (2 * k_ex) * 1e3, "paper_ms_other_hardware": paper_ms})
            del kcs, vcs
            torch.cuda.empty_cache()
        ex["flash_decoding"] = dec
        # Block-sparse attention (Section 4.3): a BigBird-like mask over 32 x 32 blocks at N = 4096 in the geometry
        # of the paper's single-GPU tables (B = 4, 12 heads, D = 64), RoPE fused, no causal rule.  Diagonal blocks,
        # one global block column and row, one seeded random block per row.  FLOPs are counted on the kept pairs.
        import numpy as _np
        nb_ = 32
        rng_ = _np.random.Generator(_np.random.PCG64(_np.random.SeedSequence([20260913, 901])))
        act = _np.eye(nb_, dtype=bool)
        act[:, 0] = True
        act[0, :] = True
        act[_np.arange(nb_), rng_.integers(0, nb_, size=nb_)] = True
        wb = synth.Workload("bigbird_d64_n4096", 4, 12, 12, 4096, 64, theta=1.0e4, causal=False, backward=True, seed_id=53)
        rb_, mb_, tbb = specs(wb)
        sb = make_sets(wb, 2)
        bmask = af.BlockMask(act, device=dev)
        ob = torch.empty((wb.B, wb.Hq, wb.S, wb.D), dtype=torch.bfloat16, device=dev)
        lb = torch.empty((wb.B, wb.Hq, wb.S), dtype=torch.float32, device=dev)
        t_bf, _, _ = timed(lambda i: af.fwd_blocks(sb[i % 2]["q"], sb[i % 2]["k"], sb[i % 2]["v"], rb_, tbb, mb_, wb.scale,
                                                   bmask, out=ob, lse=lb), k_ex, w_ex)
        t_df, _, _ = timed(lambda i: af.fwd(sb[i % 2]["q"], sb[i % 2]["k"], sb[i % 2]["v"], rb_, tbb, mb_, wb.scale, out=ob,
                                            lse=lb), k_ex, w_ex)
        af.fwd_blocks(sb[0]["q"], sb[0]["k"], sb[0]["v"], rb_, tbb, mb_, wb.scale, bmask, out=ob, lse=lb)
        wsbb = torch.empty(af.bwd_workspace_bytes(wb.B, wb.Hq, wb.Hkv, wb.S, wb.D), dtype=torch.uint8, device=dev)
        t_bb, _, _ = timed(lambda i: af.bwd(sb[0]["q"], sb[0]["k"], sb[0]["v"], ob, lb, sb[0]["do"], rb_, tbb, mb_, wb.scale,
                                            workspace=wsbb, blocks=bmask), k_ex, w_ex)
        nnz_b = int(act.sum()) * 128 * 128
        fl_b = 4.0 * wb.D * nnz_b * wb.B * wb.Hq
        ex[wb.name] = {"active_blocks": int(act.sum()), "density": float(act.mean()),
                       "fwd_ms": t_bf / k_ex, "fwd_tflops_on_kept_pairs": fl_b / (t_bf / k_ex) / 1e9,
                       "dense_fwd_ms_same_shape": t_df / k_ex, "speedup_over_dense": t_df / t_bf,
                       "bwd_ms": t_bb / k_ex, "bwd_tflops_on_kept_pairs": 2.5 * fl_b / (t_bb / k_ex) / 1e9,
                       "paper_fwd_ms_other_hardware": 0.084}
        # a second mask at the density the paper quotes (about 7.7 % of the blocks): diagonal, global block column,
        # and a seeded random block in every second row
        act2 = _np.eye(nb_, dtype=bool)
        act2[:, 0] = True
        rows2 = _np.arange(0, nb_, 2)
        act2[rows2, rng_.integers(1, nb_, size=rows2.size)] = True
        bmask2 = af.BlockMask(act2, device=dev)
        t_bf2, _, _ = timed(lambda i: af.fwd_blocks(sb[i % 2]["q"], sb[i % 2]["k"], sb[i % 2]["v"], rb_, tbb, mb_, wb.scale,
                                                    bmask2, out=ob, lse=lb), k_ex, w_ex)
        ex[wb.name]["at_paper_density"] = {"active_blocks": int(act2.sum()), "density": float(act2.mean()),
                                           "fwd_ms": t_bf2 / k_ex, "speedup_over_dense": t_df / t_bf2}
        del sb
        torch.cuda.empty_cache()
        # Rotation Calculus sweep (Section 5.3): fused vs separate RoPE at constant B*S = 32768 tokens, with the
        # hybrid arm and the same kernel without RoPE as the floor, in the Llama geometry (32 q / 8 kv heads, D = 128)
        # and in the geometry of the paper's own table (12 heads, D = 64).
        def plain_ms(wl, sets_):
            r, m, tb = specs(wl)
            oo = torch.empty((wl.B, wl.Hq, wl.S, wl.D), dtype=torch.bfloat16, device=dev)
            ll = torch.empty((wl.B, wl.Hq, wl.S), dtype=torch.float32, device=dev)
            norope = af.RopeSpec()
            t, _, _ = timed(lambda i: af.fwd(sets_[i % len(sets_)]["q"], sets_[i % len(sets_)]["k"], sets_[i % len(sets_)]["v"],
                                             norope, None, m, wl.scale, out=oo, lse=ll), k_ex, w_ex)
            return t / k_ex

        def crossover(rows):
            """S at which fused / separate crosses 1 (log-linear interpolation between neighbouring lengths)."""
            for a, b_ in zip(rows, rows[1:]):
                fa, fb_ = a["speedup_fused"] - 1.0, b_["speedup_fused"] - 1.0
                if fa == 0.0:
                    return float(a["S"])
                if fa * fb_ < 0:
                    x = fa / (fa - fb_)
                    return float(math.exp(math.log(a["S"]) + x * (math.log(b_["S"]) - math.log(a["S"]))))
            return None

        def sweep_geometry(Hq_, Hkv_, D_, theta_, tokens, lengths):
            rows = []
            for S in lengths:
                wl = synth.Workload("sweep_S%d" % S, tokens // S, Hq_, Hkv_, S, D_, theta=theta_, seed_id=50)
                ms_f, ss = fwd_ms(wl, True)
                ms_s, _ = fwd_ms(wl, False, ss)
                ms_h, _ = fwd_ms(wl, True, ss, hybrid=True)
                ms_p = plain_ms(wl, ss)
                # K-tile rotations the fused kernel performs: one per key tile and CTA (a CTA holds two query tiles:
                # two heads of a kv group when the group is even, else two consecutive row blocks of a head)
                n = (S + 127) // 128
                pair = (Hq_ // Hkv_) % 2 == 0
                rot = wl.B * (Hq_ // 2) * n * (n + 1) // 2 if pair else wl.B * Hq_ * sum(min(2 * r + 2, n) for r in range((n + 1) // 2))
                rows.append({"S": S, "B": wl.B, "fused_ms": ms_f, "separate_ms": ms_s, "hybrid_ms": ms_h, "no_rope_ms": ms_p,
                             "speedup_fused": ms_s / ms_f, "speedup_hybrid_over_fused": ms_f / ms_h,
                             "fused_tflops": wl.fwd_flops() / ms_f / 1e9, "hybrid_tflops": wl.fwd_flops() / ms_h / 1e9,
                             "no_rope_tflops": wl.fwd_flops() / ms_p / 1e9, "key_tile_rotations": rot})
                del ss
                torch.cuda.empty_cache()
            # cost of one on-chip key-tile rotation as the fused kernel pays it: least squares through the origin of
            # (fused - no RoPE) against rotations per SM
            xs = np.array([r["key_tile_rotations"] / 148.0 for r in rows])
            ys = np.array([(r["fused_ms"] - r["no_rope_ms"]) * 1e3 for r in rows])
            t_rot_us = float((xs * ys).sum() / (xs * xs).sum())
            return {"geometry": {"Hq": Hq_, "Hkv": Hkv_, "D": D_, "tokens": tokens}, "rows": rows,
                    "crossover_S": crossover(rows),
                    "t_rot_us_per_key_tile_rotation": t_rot_us,
                    "t_rot_note": "fused minus the same kernel without RoPE, per key-tile rotation and SM (it contains the "
                                  "Q rotation of the prologue and the hand-offs); the separate pass costs 4*B*S*D*(Hq+Hkv) bytes"}

        ex["rotation_calculus_sweep"] = sweep_geometry(32, 8, 128, 5.0e5, 32768, (512, 1024, 2048, 4096, 8192, 16384, 32768))
        ex["rotation_calculus_sweep_d64_h12"] = sweep_geometry(12, 12, 64, 1.0e4, 16384, (512, 1024, 2048, 4096, 8192, 16384))
        ex["rotation_calculus_ridge"] = dict(RIDGE_CONTEXT, b200_measured_flop_per_byte=peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9),
                                             paper_crossover="~5.5k tokens on H100, none on RTX 3090 (Section 5.3)")
        # separate RoPE kernel alone on a larger-than-L2 buffer (HBM roofline)
        wl = synth.CONFIGS[3]
        x = torch.randn((wl.B, wl.Hq, wl.S, wl.D), device=dev).to(torch.bfloat16)
        y = torch.empty_like(x)
        rr, _, tb = specs(wl)
        t_r, _, _ = timed(lambda i: af.rope(x, rr, tb, out=y), k_ex, w_ex)
        gbs = 2 * x.numel() * 2 / (t_r / k_ex * 1e-3) / 1e9
        ex["rope_apply_kernel"] = {"bytes": 2 * x.numel() * 2, "ms": t_r / k_ex, "GB/s": gbs,
                                   "frac_of_measured_hbm": gbs / peaks["hbm_gbs"]}
        # host time of a call through the C-ABI binding (argument marshalling, tensor-map encoding, launches), no sync
        def host_us(fn, n=200):
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for i in range(n):
                fn(i)
            dt = time.perf_counter() - t0
            torch.cuda.synchronize()
            return dt / n * 1e6
        wt = synth.Workload("host_call_probe", 1, 8, 2, 256, 128, theta=5.0e5, backward=True, seed_id=54)
        rt, mt, tt_ = specs(wt)
        st_ = make_sets(wt, 1)[0]
        ot, lt = af.fwd(st_["q"], st_["k"], st_["v"], rt, tt_, mt, wt.scale)
        wst = torch.empty(af.bwd_workspace_bytes(wt.B, wt.Hq, wt.Hkv, wt.S, wt.D), dtype=torch.uint8, device=dev)
        ex["host_us_per_call"] = {
            "fwd": host_us(lambda i: af.fwd(st_["q"], st_["k"], st_["v"], rt, tt_, mt, wt.scale, out=ot, lse=lt)),
            "bwd": host_us(lambda i: af.bwd(st_["q"], st_["k"], st_["v"], ot, lt, st_["do"], rt, tt_, mt, wt.scale, workspace=wst)),
            "decode": ex["flash_decoding"][0]["c_abi_call_from_host_us"],
            "note": "Python ctypes binding included; small shapes so that the device never back-pressures the host"}
        line["extras"] = ex
        # the three arms of the fuse-or-not experiment on the headline workload, side by side (TFLOP/s)
        c2 = ex[synth.CONFIGS[1].name]
        line["arms_on_headline_workload"] = {
            "fused_single_kernel": c2["fused_fwd_tflops"], "separate_rope_then_attention": c2["separate_rope_fwd_tflops"],
            "hybrid_k_prerotated_q_fused": c2["hybrid_fwd_tflops"],
            "hybrid_frac_of_measured_burst_peak": c2["hybrid_frac_of_measured_burst_peak"],
            "note": "value/roofline above are the single fused kernel; the other arms include their RoPE pass"}

    if rank == 0 and world == 1 and args.cpu_baseline:
        v, sample, _ = oracle_rate(w, 12.0)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": len(os.sched_getaffinity(0)), "kind": "oracle",
                                "sample": sample}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
