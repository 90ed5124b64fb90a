"""Benchmark of the UoE routed hot path: one step = one forward pass of a whole UoE block
(router -> SMHA -> router -> UoME; a block without attention or without MLP skips that half; the scale
workload adds the UoME backward) over one batch of seeded synthetic input.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2_lm] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is tokens/s with inputs resident in HBM; `e2e` is the same metric
through the public API with host buffers (pinned host -> device copy of x and device -> host copy of the
result inside the timed region).  L2 is flushed between timed steps (a 512 MB write), and every step is
timed with its own pair of CUDA events on the launching stream.  `--impl reference` times the float64
CPU oracle on the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

import uoe_inputs as gen

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------------------------
# algorithmic work per launch, by profile label
# ------------------------------------------------------------------------------------------------

def work_table(w: gen.Workload):
    s = 2 if w.dtype == "bf16" else 4
    R, d, n = w.R, w.d, w.n
    x_bytes = w.B * w.L * d * s
    t = {
        "route": dict(flops=2 * w.B * w.L_valid * d * n, bytes=w.B * w.L_valid * d * s),
        "gather": dict(flops=0, bytes=2 * R * d * s),
        "combine": dict(flops=2 * R * d, bytes=R * d * s + 2 * x_bytes),
        "plan": dict(flops=0, bytes=0),
    }
    if w.d_ff:
        de = w.d_e
        t["gemm1_act"] = dict(flops=2 * R * d * de, bytes=(R * d + R * de + n * d * de) * s)
        t["gemm2"] = dict(flops=2 * R * de * d, bytes=(R * de + R * d + n * d * de) * s)
        # both GEMMs in one kernel (narrow experts): the hidden tile is neither written nor read back
        t["mlp_fused"] = dict(flops=4 * R * d * de, bytes=(2 * R * d + 2 * n * d * de) * s)
    if w.d_ff and w.backward:
        de = w.d_e
        for name in ("bwd_da_dh", "bwd_dx", "wgrad_W1", "wgrad_W2"):
            t[name] = dict(flops=2 * R * d * de, bytes=(R * d + 2 * R * de + n * d * de) * s)
        t["wgrad_W1"]["bytes"] = t["wgrad_W2"]["bytes"] = (R * d + R * de) * s + n * d * de * 4
        t["pool"] = dict(flops=0, bytes=x_bytes)
    if w.H:
        dg = w.d_g
        att = 4 * w.l_a * w.l_a * dg * w.B * w.k
        att = att // 2 if w.causal else att
        t["qkv_proj"] = dict(flops=6 * R * d * dg, bytes=(R * d + 3 * R * dg + 3 * n * d * dg) * s)
        t["attention"] = dict(flops=att, bytes=4 * R * dg * s)
        t["out_proj"] = dict(flops=2 * R * dg * d, bytes=(R * dg + R * d + n * dg * d) * s)
    if w.H and w.backward:
        # algorithmic work of the attention backward is five l_a x l_a contractions (dV, dP, dK, dQ and the
        # rebuilt S); the dK/dV pass is credited with four of them, the dQ pass with one
        t["attn_bwd_dkdv"] = dict(flops=2 * att, bytes=6 * R * dg * s)
        t["attn_bwd_dq"] = dict(flops=att // 2, bytes=5 * R * dg * s)
        t["bwd_do"] = dict(flops=2 * R * d * dg, bytes=(R * d + R * dg + n * dg * d) * s)
        t["wgrad_Wo"] = dict(flops=2 * R * d * dg, bytes=(R * d + R * dg) * s + n * d * dg * 4)
        t["wgrad_Wqkv"] = dict(flops=6 * R * d * dg, bytes=(R * d + 3 * R * dg) * s + 3 * n * d * dg * 4)
        t["bwd_dx_att"] = dict(flops=6 * R * dg * d, bytes=(3 * R * dg + R * d + 3 * n * d * dg) * s)
    return t


def step_flops(w: gen.Workload) -> int:
    t = work_table(w)
    f = 0
    if w.d_ff:
        f += t["gemm1_act"]["flops"] + t["gemm2"]["flops"]
    if w.d_ff and w.backward:
        f += sum(t[k]["flops"] for k in ("bwd_da_dh", "bwd_dx", "wgrad_W1", "wgrad_W2"))
    if w.H:
        f += t["qkv_proj"]["flops"] + t["attention"]["flops"] + t["out_proj"]["flops"]
    if w.H and w.backward:
        f += t["attn_bwd_dkdv"]["flops"] + t["attn_bwd_dq"]["flops"] + t["bwd_do"]["flops"] + t["wgrad_Wo"]["flops"] + \
            t["wgrad_Wqkv"]["flops"] + t["bwd_dx_att"]["flops"]
    return f


# ------------------------------------------------------------------------------------------------
# inputs
# ------------------------------------------------------------------------------------------------

def host_inputs(w: gen.Workload):
    d = dict(x=gen.make_x(w))
    if w.H:
        d["Wr_att"] = gen.make_router(w, "att")
        d["Wq"], d["Wk"], d["Wv"], d["Wo"] = gen.make_attn_weights(w)
    if w.d_ff:
        d["Wr_mlp"] = gen.make_router(w, "mlp")
        d["W1"], d["W2"] = gen.make_mlp_weights(w)
    if w.backward:
        d["dy"] = gen.make_dy(w)
    return d


def oracle_step(w: gen.Workload, h, B=None):
    """One block forward with the float64 oracle on the first B samples; returns seconds."""
    from oracle import uoe_oracle as orc
    B = w.B if B is None else B
    x = h["x"].f64[:B]
    t0 = time.perf_counter()
    cur = x
    if w.H:
        r_att = orc.route(cur, h["Wr_att"].f64, w.k, w.m, w.c, L_valid=w.L_valid)
        cur = orc.smha_forward(cur, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, r_att, w.d_h, w.causal)
    if w.d_ff:
        r = orc.route(cur, h["Wr_mlp"].f64, w.k, w.m, w.c, L_valid=w.L_valid)
        u = cur
        cur = orc.mlp_forward(u, h["W1"].f64, h["W2"].f64, r, w.act)
        if w.backward:
            g = orc.mlp_backward(u, h["W1"].f64, h["W2"].f64, h["Wr_mlp"].f64, r, h["dy"].f64[:B], w.act)[0]
    elif w.backward:
        g = h["dy"].f64[:B]
    if w.H and w.backward:
        orc.smha_backward(x, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, h["Wr_att"].f64, r_att, g, w.d_h, w.causal)
    return time.perf_counter() - t0


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        ns = [p.get("num_threads", 1) for p in threadpool_info()]
        return max(ns) if ns else 1
    except Exception:
        return os.cpu_count() or 1


def cpu_sample_B(w: gen.Workload) -> int:
    """Samples of the workload the oracle is timed on: sized for seconds, not minutes."""
    per_sample_gflop = step_flops(w) / w.B / 1e9
    budget_gflop = 40.0            # roughly 1-3 s of float64 work per step on a few host cores
    return max(1, min(w.B, int(budget_gflop / max(per_sample_gflop, 1e-9))))


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------

class ClockSampler:
    """SM clock and clock-event reasons of one GPU, read (never set) through NVML from a background thread
    every few milliseconds while the timed region runs."""

    def __init__(self, torch_device_index: int, period_s: float = 0.005):
        import threading
        self.period = period_s
        self.sm, self.reasons, self.power = [], set(), []
        self.sm_max = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            h = None
            try:
                uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
                h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode() if not uuid.startswith("GPU-") else uuid.encode())
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self._h = h
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _sample(self):
        nv, h = self._nv, self._h
        self.sm.append(float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
        r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
        for name, bit in (("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown),
                          ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                          ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown),
                          ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap)):
            if r & bit:
                self.reasons.add(name)
        try:
            self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            try:
                self._sample()
            except Exception:
                break
            self._stop.wait(self.period)

    def start(self):
        if self._h is None:
            return
        import threading
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": []}
        if self._thread is None:
            return out
        try:
            self._sample()          # at least one reading taken while the last timed kernels are in flight
        except Exception:
            pass
        self._stop.set()
        self._thread.join(timeout=2)
        if self.sm:
            out = {"sm_mhz": statistics.median(self.sm), "sm_min_mhz": min(self.sm), "sm_max_mhz": self.sm_max,
                   "reasons": sorted(self.reasons), "samples": len(self.sm),
                   "power_w_max": max(self.power) if self.power else None, "source": "nvml"}
        return out


# ------------------------------------------------------------------------------------------------
# arms
# ------------------------------------------------------------------------------------------------

def base_line(w: gen.Workload, args, n_gpus: int):
    return {
        "metric": "UoME+SMHA layer tokens/s", "unit": "tokens/s", "n_gpus": n_gpus, "steps": args.steps,
        "warmup": args.warmup, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": w.name, "stands_in_for": w.stands_in_for, "B": w.B, "L": w.L, "L_valid": w.L_valid,
                   "d": w.d, "n": w.n, "k": w.k, "m": w.m, "c": w.c, "d_ff": w.d_ff, "heads": w.H, "d_h": w.d_h,
                   "causal": w.causal, "act": w.act, "blocks": ("smha+" if w.H else "") + ("uome" if w.d_ff else "") + ("+backward" if w.backward else ""),
                   "parallelism": f"replicas x{n_gpus}" if n_gpus > 1 else "single gpu",
                   "l2": "flushed between timed steps (512 MB write)"},
    }


def max_over_ranks(values, world: int, device=None):
    """Element-wise max of a list of floats over all ranks (the job is as slow as its slowest replica)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(w: gen.Workload, world: int, ms_per_step: float) -> float:
    """Whole-job tokens/s of `world` replicas that each process the workload once per step."""
    return w.B * w.L_valid * world / (ms_per_step * 1e-3)


def run_reference(args, w: gen.Workload, rank: int, world: int):
    if rank != 0:
        return
    h = host_inputs(w)
    Bs = cpu_sample_B(w)
    for _ in range(args.warmup):
        oracle_step(w, h, Bs)
    ts = [oracle_step(w, h, Bs) for _ in range(args.steps)]
    sec = sum(ts) / len(ts)
    tok_s = Bs * w.L_valid / sec
    line = base_line(w, args, 1)
    line.update({"impl": "reference", "value": tok_s, "ms_per_step": sec * 1e3, "dtype": "f64", "n_gpus": world,
                 "tflops": step_flops(w) * Bs / w.B / sec / 1e12,
                 "cpu_baseline": {"value": tok_s, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                                  "sample": f"first {Bs} of {w.B} samples, whole block, {args.steps} steps"},
                 "e2e": {"value": tok_s, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                 "gpu_launches": 0})
    print(json.dumps(line), flush=True)


def measure_gpu(args, w: gen.Workload, dev, world: int, steps: int, warmup: int, with_e2e: bool):
    """Times `steps` steps of workload w on this rank's GPU.  Returns a dict with the per-step milliseconds
    (device events, L2 flushed between steps), launches, clocks, per-kernel records and the e2e time."""
    import torch

    import paper_2503_02495_b200 as uoe
    from paper_2503_02495_b200.block import UoEBlock
    from paper_2503_02495_b200.workload import problem_of, to_dev

    h = host_inputs(w)
    wd = {k: to_dev(v, dev) for k, v in h.items() if k not in ("x", "dy")}
    x_dev = to_dev(h["x"], dev)
    dy_dev = to_dev(h["dy"], dev) if w.backward else None
    blk = UoEBlock(problem_of(w, "att") if w.H else None, problem_of(w, "mlp") if w.d_ff else None, wd, dev,
                   backward=w.backward)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step(xin):
        if args.part == "route":          # the router alone (profiling): one uoe_route call on the block's input
            if blk.pm is not None:
                uoe.uoe_route(blk.pm, xin, wd["Wr_mlp"], out=blk.rm, ws=blk.ws_rm, check=False)
                return blk.rm.gate
            uoe.uoe_route(blk.pa, xin, wd["Wr_att"], out=blk.ra, ws=blk.ws_ra, check=False)
            return blk.ra.gate
        out = blk.forward(xin)
        if w.backward:
            g = dy_dev
            if w.d_ff:
                blk.mlp_backward(blk.u if w.H else xin, g)
                g = blk.dx
            if w.H:
                blk.smha_backward(xin, g)
                g = blk.dh
            return g
        return out

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(warmup, 3)):
        step(x_dev)
    torch.cuda.synchronize()
    st = blk.device_status()
    if st != 0:
        raise RuntimeError("device status after warm-up: " + uoe.status_string(st))

    # ---- timed region: K steps, each with its own event pair, L2 flushed in between ----
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier()
    launches0 = uoe.uoe_launch_count()
    for e0, e1 in ev:
        flush.zero_()
        e0.record(stream)
        step(x_dev)
        e1.record(stream)
    barrier()
    launches = uoe.uoe_launch_count() - launches0
    clocks = sampler.stop()
    ms = [e0.elapsed_time(e1) for e0, e1 in ev]
    res = {"ms_step": sum(ms) / len(ms), "ms_min": min(ms), "launches": int(launches), "clocks": clocks, "host": h}

    # ---- end to end through the public API with host buffers ----
    if with_e2e:
        x_host = h["x"].raw
        x_pin = torch.from_numpy(np.ascontiguousarray(x_host).view(np.int16 if w.dtype == "bf16" else np.float32)).pin_memory()
        x_in = torch.empty_like(x_dev)
        y_pin = torch.empty(x_pin.shape, dtype=x_pin.dtype).pin_memory()
        e2e_t = []
        for i in range(steps + 2):
            flush.zero_()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            x_in.view(x_pin.dtype).copy_(x_pin, non_blocking=True)
            out = step(x_in)
            if out.shape == x_in.shape:
                y_pin.copy_(out.view(x_pin.dtype), non_blocking=True)
            torch.cuda.synchronize()
            if i >= 2:
                e2e_t.append(time.perf_counter() - t0)
        res["e2e_ms"] = sum(e2e_t) / len(e2e_t) * 1e3
        res["h2d"] = int(x_pin.numel() * x_pin.element_size())
        res["d2h"] = int(y_pin.numel() * y_pin.element_size())

    # ---- per-kernel durations (separate pass: the event pairs would perturb the timed region) ----
    steps_prof = min(steps, 20)
    uoe.uoe_profile_enable(True)
    for _ in range(steps_prof):
        flush.zero_()
        step(x_dev)
    torch.cuda.synchronize()
    uoe.uoe_profile_enable(False)
    per = {}
    for name, t in uoe.uoe_profile_records():
        per.setdefault(name, []).append(t)
    work = work_table(w)
    tot = sum(sum(v) for v in per.values())
    kern = []
    for name, v in per.items():
        avg = sum(v) / len(v)
        wk = work.get(name, dict(flops=0, bytes=0))
        kern.append({"kernel": name, "launches_per_step": len(v) / steps_prof, "avg_ms": avg,
                     "share": sum(v) / tot if tot else 0.0,
                     "tflops": wk["flops"] / avg / 1e9 if avg > 0 else 0.0,
                     "gbs": wk["bytes"] / avg / 1e6 if avg > 0 else 0.0})
    kern.sort(key=lambda r: -r["share"])
    res["kernels"] = kern
    del blk, flush
    torch.cuda.empty_cache()
    return res


TENSOR_KERNELS = ("gemm1_act", "gemm2", "mlp_fused", "qkv_proj", "out_proj", "attention", "bwd_da_dh", "bwd_dx", "wgrad_W1", "wgrad_W2",
                  "attn_bwd_dkdv", "attn_bwd_dq", "bwd_do", "bwd_dx_att", "wgrad_Wo", "wgrad_Wqkv")
HBM_KERNELS = ("route", "gather", "combine", "pool")


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/
# (step_kernels_cfg2_lm.md, launches_gemm_cfg5_scale_B4.md, route_kernels_cfg5_scale.md).  Keyed by (workload, kernel
# label); an entry is dropped when its kernel changes, and the line then reports null.  The scale workload's GEMM
# entries were captured at B=4 and scaled by 2 (the part that is weight reads does not grow with B, so they are upper
# estimates); its route entry was captured at full size.
NCU_TRAFFIC = {
    ("cfg2_lm", "route"): 8.47e6,
    ("cfg2_lm", "combine"): 25.18e6,
    ("cfg2_lm", "qkv_proj"): 9.73e6,
    ("cfg2_lm", "mlp_fused"): 12.34e6,
    ("cfg2_lm", "attention"): 6.88e6,
    ("cfg5_scale", "gemm1_act"): 2 * (351.9e6 + 105.7e6),
    ("cfg5_scale", "gemm2"): 2 * (176.2e6 + 220.0e6),
    ("cfg5_scale", "bwd_da_dh"): 2 * (442.7e6 + 113.8e6),
    ("cfg5_scale", "bwd_dx"): 2 * (176.3e6 + 220.6e6),
    ("cfg5_scale", "route"): 268.4e6 + 16.8e6,
}


def roofline_of(top, w: gen.Workload, peaks, peak_src):
    wk = work_table(w).get(top["kernel"], dict(flops=0, bytes=0))
    t_tensor = wk["flops"] / (peaks["bf16_tflops"] * 1e12)
    t_hbm = wk["bytes"] / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm and wk["flops"] > 0:
        roof = {"bound": "tensor", "achieved": top["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": top["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": NCU_TRAFFIC.get((w.name, top["kernel"])),
                 "kernel": top["kernel"],
                 "avg_ms": top["avg_ms"], "share_of_kernel_time": top["share"], "peak_source": peak_src,
                 "algorithmic_flops": wk["flops"], "algorithmic_bytes": wk["bytes"]})
    return roof


def run_ours(args, w: gen.Workload, rank: int, local_rank: int, world: int):
    import torch
    import torch.distributed as dist

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    m = measure_gpu(args, w, dev, world, args.steps, args.warmup, True)
    ms_step, e2e_ms = max_over_ranks([m["ms_step"], m["e2e_ms"]], world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_src = load_peaks()
    tokens = w.B * w.L_valid * world
    flops = step_flops(w) * world
    kern = m["kernels"]
    roof = roofline_of(kern[0], w, peaks, peak_src)

    # ---- CPU baseline: the oracle as it stands, on a bounded sample ----
    h = m["host"]
    Bs = cpu_sample_B(w)
    ts = []
    if not args.skip_cpu_baseline:
        oracle_step(w, h, Bs)
        t_begin = time.perf_counter()
        while len(ts) < 3 or (time.perf_counter() - t_begin < 8.0 and len(ts) < 20):
            ts.append(oracle_step(w, h, Bs))
    cpu_sec = sum(ts) / len(ts) if ts else float("nan")

    line = base_line(w, args, world)
    line.update({
        "value": job_throughput(w, world, ms_step), "ms_per_step": ms_step, "ms_per_step_min": m["ms_min"],
        "tflops": flops / (ms_step * 1e-3) / 1e12,
        "frac_of_bf16_peak": flops / (ms_step * 1e-3) / 1e12 / (peaks["bf16_tflops"] * world),
        "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"]},
        "gpu_launches": m["launches"],
        "clocks": m["clocks"],
        "roofline": roof,
        "kernels": kern,
        "cpu_baseline": {"value": (Bs * w.L_valid / cpu_sec) if ts else None, "unit": "tokens/s", "cores": blas_threads(),
                         "kind": "oracle", "sec_per_step": cpu_sec if ts else None,
                         "sample": f"first {Bs} of {w.B} samples, whole block, {len(ts)} steps"},
    })
    del m, h

    # ---- the large MLP workload (forward + backward), where the tensor-core and HBM targets are quoted ----
    if world == 1 and not args.no_scale and w.name != "cfg5_scale" and args.B == 0:
        ws = gen.WORKLOADS["cfg5_scale"]
        ms5 = measure_gpu(args, ws, dev, 1, 10, 3, False)
        k5 = {r["kernel"]: r for r in ms5["kernels"]}
        tens = [k5[n] for n in TENSOR_KERNELS if n in k5]
        wt = work_table(ws)
        tf_sum = sum(wt[r["kernel"]]["flops"] for r in tens)
        tm_sum = sum(r["avg_ms"] * r["launches_per_step"] for r in tens)
        line["scale_workload"] = {
            "workload": ws.name, "blocks": "uome forward + backward", "B": ws.B, "L": ws.L, "d": ws.d, "d_ff": ws.d_ff,
            "n": ws.n, "k": ws.k, "m": ws.m, "c": ws.c, "steps": 10,
            "ms_per_step": ms5["ms_step"], "tokens_per_s": ws.B * ws.L_valid / (ms5["ms_step"] * 1e-3),
            "tflops": step_flops(ws) / (ms5["ms_step"] * 1e-3) / 1e12,
            "frac_of_bf16_peak": step_flops(ws) / (ms5["ms_step"] * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "grouped_gemm_tflops": tf_sum / tm_sum / 1e9 if tm_sum > 0 else None,
            "grouped_gemm_frac_of_bf16_peak": tf_sum / tm_sum / 1e9 / peaks["bf16_tflops"] if tm_sum > 0 else None,
            "hbm_kernels": {n: {"gbs": k5[n]["gbs"], "frac_of_hbm_peak": k5[n]["gbs"] / peaks["hbm_gbs"]}
                            for n in HBM_KERNELS if n in k5},
            "gpu_launches": ms5["launches"], "clocks": ms5["clocks"],
            "roofline": roofline_of(ms5["kernels"][0], ws, peaks, peak_src),
            "kernels": [{kk: (round(vv, 5) if isinstance(vv, float) else vv) for kk, vv in r.items()} for r in ms5["kernels"]],
        }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2_lm", choices=sorted(gen.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--B", type=int, default=0, help="override the workload's batch size (profiling on a smaller case)")
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="omit the oracle timing (profiling runs)")
    ap.add_argument("--backward", action="store_true", help="add the backward of every half of the block to the step")
    ap.add_argument("--part", default="all", choices=["all", "route"], help="time only a part of the step (profiling runs)")
    ap.add_argument("--no-scale", action="store_true", help="do not add the scale workload's summary to the line")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    w = gen.WORKLOADS[args.workload]
    if args.B > 0:
        w = w.replace(B=args.B)
    if args.backward:
        w = w.replace(backward=True)
    if args.impl == "reference":
        run_reference(args, w, rank, world)
    else:
        run_ours(args, w, rank, local_rank, world)


if __name__ == "__main__":
    main()
