"""Benchmark of the UoE routed hot path.  One step = one pass of the whole hot path over one batch of seeded
synthetic input: router -> SMHA -> router -> UoME for a block workload (a block without attention or without MLP
skips that half), router -> UoME forward -> UoME backward for the scale workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5_scale] [--impl ours|reference]

Prints ONE JSON line (rank 0).  The top-level keys describe the largest single-GPU workload (cfg5_scale); with one
GPU the line also carries, under "workloads", one block per other workload (language-model, long-sequence, image and
the small float32 shape) measured with the same protocol: step time, tokens/s, TFLOP/s, roofline of the dominant
kernel, the oracle's CPU time on a bounded sample, and parity statistics against the oracle (max error over
tolerance, near-tie index mismatches).  `value` is tokens/s with inputs resident in HBM; `e2e` is the same metric
through the public API with host buffers (pinned host -> device copies of the step's inputs and a device -> host
copy of its result inside the timed region).  Small workloads: L2 is flushed between timed steps (a 512 MB write)
and every step has its own pair of CUDA events; the scale workload streams far more than L2 per step and is timed
back to back, once for K steps and once for at least a second ("sustained", against the sustained peak).
`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
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

def patch_major(w: gen.Workload) -> bool:
    """Whether the library runs the second expert layer (and the backward's dx) walked by output patch, combine
    included: bfloat16, patches of 128 tokens, 256-column output tiles, experts wider than the one-kernel MLP takes."""
    return bool(w.d_ff) and w.dtype == "bf16" and w.L // w.m == 128 and w.d % 256 == 0 and w.d_e % 64 == 0 and \
        not (w.d_e == 256 and w.d <= 512) and w.k <= 8


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
        if patch_major(w):    # second layer and combine in one kernel: reads a', W2 and x, writes y (no z)
            t["gemm2"] = dict(flops=2 * R * de * d, bytes=(R * de + n * d * de) * s + 2 * x_bytes)
    if w.d_ff and w.backward:
        de = w.d_e
        for name in ("bwd_da_dh", "bwd_dx", "wgrad_W1", "wgrad_W2"):
            t[name] = dict(flops=2 * R * d * de, bytes=(R * d + 2 * R * de + n * d * de) * s)
        t["wgrad_W1"]["bytes"] = t["wgrad_W2"]["bytes"] = (R * d + R * de) * s + n * d * de * 4
        if patch_major(w):    # dx_g and the backward combine in one kernel: reads dh, W1 and dy, writes dx
            t["bwd_dx"] = dict(flops=2 * R * d * de, bytes=(R * de + n * d * de) * s + 2 * x_bytes)
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

TOP_WORKLOAD = "cfg5_scale"          # the largest single-GPU workload: the one the headline line sits on
ALL_WORKLOADS = ("cfg1_small_f32", "cfg2_lm", "cfg3_long", "cfg4_vit", "cfg5_scale")
L2_BYTES = 126 << 20


def config_of(w: gen.Workload, n_gpus: int, l2: str):
    return {"workload": w.name, "stands_in_for": w.stands_in_for, "B": w.B, "L": w.L, "L_valid": w.L_valid,
            "d": w.d, "n": w.n, "k": w.k, "m": w.m, "c": w.c, "d_ff": w.d_ff, "heads": w.H, "d_h": w.d_h,
            "causal": w.causal, "act": w.act,
            "blocks": ("smha+" if w.H else "") + ("uome" if w.d_ff else "") + ("+backward" if w.backward else ""),
            "parallelism": f"replicas x{n_gpus}" if n_gpus > 1 else "single gpu", "l2": l2}


def base_line(w: gen.Workload, args, n_gpus: int, l2: str = "flushed between timed steps (512 MB write)"):
    return {
        "metric": "UoME+SMHA layer tokens/s", "unit": "tokens/s", "n_gpus": n_gpus, "steps": args.steps,
        "warmup": args.warmup, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": w.dtype, "data": "synthetic", "config": config_of(w, n_gpus, l2),
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


def inputs_exceed_l2(w: gen.Workload) -> bool:
    """True when one step streams far more than the L2 holds, so that no step finds its inputs cached."""
    s = 2 if w.dtype == "bf16" else 4
    return w.B * w.L * w.d * s >= 2 * L2_BYTES


def cpu_baseline_of(w: gen.Workload, h, budget_s: float = 6.0, max_steps: int = 10):
    """The oracle as it stands, timed on the host cores on the first Bs samples of the workload."""
    Bs = cpu_sample_B(w)
    oracle_step(w, h, Bs)                                   # first call pays imports and page faults
    ts, t_begin = [], time.perf_counter()
    while len(ts) < 2 or (time.perf_counter() - t_begin < budget_s and len(ts) < max_steps):
        ts.append(oracle_step(w, h, Bs))
    sec = sum(ts) / len(ts)
    return {"value": Bs * w.L_valid / sec, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
            "sec_per_step": sec, "tflops": step_flops(w) * Bs / w.B / sec / 1e12,
            "sample": f"first {Bs} of {w.B} samples, whole step ({config_of(w, 1, '')['blocks']}), {len(ts)} steps"}


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
    line = base_line(w, args, 1, "not applicable (CPU)")
    line.update({"impl": "reference", "value": tok_s, "ms_per_step": sec * 1e3, "dtype": "f64", "n_gpus": world,
                 "tflops": step_flops(w) * Bs / w.B / sec / 1e12,
                 "cpu_baseline": {"value": tok_s, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle",
                                  "sample": f"first {Bs} of {w.B} samples, whole step, {args.steps} steps"},
                 "e2e": {"value": tok_s, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                 "gpu_launches": 0})
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# parity of the launch configuration that is timed, on a bounded sample the oracle can afford
# ------------------------------------------------------------------------------------------------

def parity_of(w: gen.Workload, h, wd, x_dev, dy_dev, dev):
    """Runs every half of the block once more through the C ABI (expert terms: residual off) and compares the first
    Bs samples with the float64 oracle fed the same stored inputs.  Returns max error over tolerance per output,
    routing-probability errors and the near-tie index mismatch counts."""
    import torch

    import paper_2503_02495_b200 as uoe
    from oracle import uoe_oracle as orc
    from paper_2503_02495_b200.workload import problem_of

    tol = 2e-2 if w.dtype == "bf16" else 1e-4
    Bs = min(cpu_sample_B(w), 64)
    f64 = lambda t: t.detach().to(torch.float64).cpu().numpy()
    rel = lambda got, ref: float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-300))
    out = {"tolerance": tol, "sample": f"first {Bs} of {w.B} samples", "outputs": {}, "routing": {}}
    worst = 0.0

    def routing_stats(tag, r_gpu, x64, Wr64):
        ro = orc.route(x64, Wr64, w.k, w.m, w.c, L_valid=w.L_valid)
        e_gpu, p_gpu = r_gpu.expert_idx[:Bs].cpu().numpy(), r_gpu.patch_idx[:Bs].cpu().numpy()
        near_e = near_p = hard = 0
        for b in range(Bs):
            if not np.array_equal(e_gpu[b], ro.expert_idx[b]):
                near_e += 1
                hard += ro.expert_margin[b] > 1e-5
                continue
            for s in range(w.k):
                if not np.array_equal(p_gpu[b, s], ro.patch_idx[b, s]):
                    near_p += 1
                    hard += ro.patch_margin[b, s] > 1e-5
        out["routing"][tag] = {
            "p_samp_max_abs_err": float(np.abs(r_gpu.p_samp[:Bs].cpu().numpy() - ro.p_samp).max()),
            "p_patch_max_abs_err": float(np.abs(r_gpu.p_patch[:Bs].cpu().numpy() - ro.p_patch).max()),
            "near_tie_expert_set_mismatches": int(near_e), "near_tie_patch_set_mismatches": int(near_p),
            "mismatches_outside_1e-5_margin": int(hard)}
        return e_gpu, p_gpu, int(hard)

    cur, cur64 = x_dev, h["x"].f64[:Bs]
    hard_total = 0
    if w.H:
        pa = problem_of(w, "att")
        r = uoe.uoe_route(pa, cur, wd["Wr_att"])
        e_gpu, p_gpu, hard = routing_stats("smha", r, cur64, h["Wr_att"].f64)
        hard_total += hard
        z = uoe.uoe_smha_forward(problem_of(w, "att", residual=False), cur, wd["Wq"], wd["Wk"], wd["Wv"], wd["Wo"], r)
        ro = orc.with_selection(cur64, h["Wr_att"].f64, e_gpu, p_gpu, w.m, w.L_valid)
        ref = orc.smha_forward(cur64, h["Wq"].f64, h["Wk"].f64, h["Wv"].f64, h["Wo"].f64, ro, w.d_h, w.causal, residual=False)
        out["outputs"]["smha_expert_term"] = rel(f64(z[:Bs]), ref) / tol
        cur = uoe.uoe_smha_forward(pa, cur, wd["Wq"], wd["Wk"], wd["Wv"], wd["Wo"], r)
        cur64 = f64(cur[:Bs])              # the UoME half is checked on the bits the GPU feeds it
    if w.d_ff:
        pm = problem_of(w, "mlp")
        r = uoe.uoe_route(pm, cur, wd["Wr_mlp"])
        e_gpu, p_gpu, hard = routing_stats("uome", r, cur64, h["Wr_mlp"].f64)
        hard_total += hard
        pm0 = problem_of(w, "mlp", residual=False)
        sh = uoe.alloc_saved_h(pm0, dev) if w.backward else None
        z = uoe.uoe_mlp_forward(pm0, cur, wd["W1"], wd["W2"], r, saved_h=sh)
        ro = orc.with_selection(cur64, h["Wr_mlp"].f64, e_gpu, p_gpu, w.m, w.L_valid)
        ref = orc.mlp_forward(cur64, h["W1"].f64, h["W2"].f64, ro, w.act, residual=False)
        out["outputs"]["uome_expert_term"] = rel(f64(z[:Bs]), ref) / tol
        if w.backward:
            dx = uoe.uoe_mlp_backward(pm0, cur, wd["W1"], wd["W2"], wd["Wr_mlp"], r, sh, dy_dev)[0]
            dref = orc.mlp_backward(cur64, h["W1"].f64, h["W2"].f64, h["Wr_mlp"].f64, ro, h["dy"].f64[:Bs], w.act,
                                    residual=False)[0]
            out["outputs"]["uome_dx_expert_term"] = rel(f64(dx[:Bs]), dref) / tol
            out["note"] = "dW1, dW2, dW_r need every sample: checked at full size in tests/test_gpu_scale.py"
            del dx, sh
    worst = max(out["outputs"].values()) if out["outputs"] else 0.0
    out["max_err_over_tol"] = worst
    out["ok"] = bool(worst <= 1.0 and hard_total == 0)
    return out


# ------------------------------------------------------------------------------------------------
# measurement of one workload on this rank's GPU
# ------------------------------------------------------------------------------------------------

def measure_gpu(args, w: gen.Workload, dev, world: int, steps: int, warmup: int, with_e2e: bool, with_parity: bool = False,
                sustain_s: float = 0.0):
    """Times `steps` steps of workload w on this rank's GPU.  Returns a dict with the step time (device events),
    launches, clocks, per-kernel records, the e2e time and, on request, the parity block and a sustained run."""
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
    big = inputs_exceed_l2(w)
    flush = None if big else torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step(xin, dyin=None):
        if args.part == "route":          # the router alone (profiling): one uoe_route call on the block's input
            if blk.pm is not None:
                uoe.uoe_route(blk.pm, xin, wd["Wr_mlp"], out=blk.rm, ws=blk.ws_rm, check=False)
                return blk.rm.gate
            uoe.uoe_route(blk.pa, xin, wd["Wr_att"], out=blk.ra, ws=blk.ws_ra, check=False)
            return blk.ra.gate
        out = blk.forward(xin)
        if w.backward:
            g = dy_dev if dyin is None else dyin
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

    def check_status(where):
        st = blk.device_status()
        if st != 0:
            raise RuntimeError(f"device status after {where}: " + uoe.status_string(st))

    for _ in range(max(warmup, 3)):
        step(x_dev)
    torch.cuda.synchronize()
    check_status("warm-up")

    # ---- timed region: K steps.  Small inputs: each step has its own event pair and L2 is flushed in between.
    #      Inputs far larger than L2: the K steps run back to back inside one event pair. ----
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    barrier()
    launches0 = uoe.uoe_launch_count()
    if big:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            step(x_dev)
        e1.record(stream)
        barrier()
        ms = [e0.elapsed_time(e1) / steps]
    else:
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for e0, e1 in ev:
            flush.zero_()
            e0.record(stream)
            step(x_dev)
            e1.record(stream)
        barrier()
        ms = [e0.elapsed_time(e1) for e0, e1 in ev]
    launches = uoe.uoe_launch_count() - launches0
    clocks = sampler.stop()
    check_status("the timed region")
    res = {"ms_step": sum(ms) / len(ms), "ms_min": min(ms), "launches": int(launches), "clocks": clocks, "host": h,
           "l2": "inputs far larger than L2 (x alone is %d MB): steps run back to back, no flush" % (w.B * w.L * w.d * 2 >> 20)
                 if big else "flushed between timed steps (512 MB write)"}

    # ---- a run long enough for the power cap to settle (same step, back to back, one event pair) ----
    if sustain_s > 0 and big:
        n_sus = max(steps, int(sustain_s * 1e3 / res["ms_step"]) + 1)
        sampler = ClockSampler(dev.index or 0, period_s=0.02)
        sampler.start()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n_sus):
            step(x_dev)
        e1.record(stream)
        torch.cuda.synchronize()
        res["sustained"] = {"steps": n_sus, "seconds": e0.elapsed_time(e1) * 1e-3, "ms_per_step": e0.elapsed_time(e1) / n_sus,
                            "clocks": sampler.stop()}
        check_status("the sustained run")

    # ---- end to end through the public API with host buffers: inputs (x, and dy when the step has a backward) from
    #      pinned host memory, the step's result back to pinned host memory, all inside the timed region ----
    if with_e2e:
        npdt = np.int16 if w.dtype == "bf16" else np.float32
        pin = lambda st: torch.from_numpy(np.ascontiguousarray(st.raw).view(npdt)).pin_memory()
        x_pin = pin(h["x"])
        x_in = torch.empty_like(x_dev)
        dy_pin = pin(h["dy"]) if w.backward else None
        dy_in = torch.empty_like(dy_dev) if w.backward else None
        y_pin = torch.empty(x_pin.shape, dtype=x_pin.dtype).pin_memory()
        e2e_t = []
        n_e2e = min(steps, 20) + 2
        for i in range(n_e2e):
            if flush is not None:
                flush.zero_()
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            x_in.view(x_pin.dtype).copy_(x_pin, non_blocking=True)
            if w.backward:
                dy_in.view(dy_pin.dtype).copy_(dy_pin, non_blocking=True)
            out = step(x_in, dy_in)
            if out.shape == x_in.shape:
                y_pin.copy_(out.view(x_pin.dtype), non_blocking=True)
            torch.cuda.synchronize()
            if i >= 2:
                e2e_t.append(time.perf_counter() - t0)
        res["e2e_ms"] = sum(e2e_t) / len(e2e_t) * 1e3
        res["e2e_steps"] = len(e2e_t)
        res["h2d"] = int(x_pin.numel() * x_pin.element_size()) * (2 if w.backward else 1)
        res["d2h"] = int(y_pin.numel() * y_pin.element_size())
        check_status("the end-to-end loop")
        del x_pin, y_pin, x_in, dy_pin, dy_in

    # ---- per-kernel durations (separate pass: the event pairs would perturb the timed region) ----
    steps_prof = min(steps, 20)
    uoe.uoe_profile_enable(True)
    for _ in range(steps_prof):
        if flush is not None:
            flush.zero_()
        step(x_dev)
    torch.cuda.synchronize()
    uoe.uoe_profile_enable(False)
    check_status("the per-kernel pass")
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
    # the whole router call (Eq. 13-14, 21 and the selection), timed by itself as it runs in a stream: CUDA events around
    # uoe_route calls on the block's input (inputs larger than L2: 20 calls back to back in one event pair; small
    # inputs: one event pair per call, L2 flushed before each).  "kernels_ms" is the sum of the per-kernel event pairs
    # of the pass above, which keeps the call's kernels from overlapping and so reads higher.
    route_labels = [n for n in per if n in ("route", "route_select")]
    t_route = sum(sum(per[n]) for n in route_labels) / steps_prof
    n_route = (1 if w.H else 0) + (1 if w.d_ff else 0)
    if t_route > 0 and n_route:
        rp, rw, rr, rws = (blk.pm, wd["Wr_mlp"], blk.rm, blk.ws_rm) if blk.pm is not None else (blk.pa, wd["Wr_att"], blk.ra, blk.ws_ra)
        for _ in range(3):
            uoe.uoe_route(rp, x_dev, rw, out=rr, ws=rws, check=False)
        torch.cuda.synchronize()
        n_calls = 20
        if big:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n_calls):
                uoe.uoe_route(rp, x_dev, rw, out=rr, ws=rws, check=False)
            e1.record(stream)
            torch.cuda.synchronize()
            ms_call = e0.elapsed_time(e1) / n_calls
        else:
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_calls)]
            for e0, e1 in ev:
                flush.zero_()
                e0.record(stream)
                uoe.uoe_route(rp, x_dev, rw, out=rr, ws=rws, check=False)
                e1.record(stream)
            torch.cuda.synchronize()
            ms_call = sum(e0.elapsed_time(e1) for e0, e1 in ev) / n_calls
        check_status("the router timing")
        res["route_call"] = {"ms": ms_call, "gbs": work["route"]["bytes"] / ms_call / 1e6, "calls": n_calls,
                             "kernels_ms": t_route / n_route, "kernels": sorted(route_labels)}
    if with_parity:
        res["parity"] = parity_of(w, h, wd, x_dev, dy_dev, dev)
    del blk, flush
    torch.cuda.empty_cache()
    return res


def single_mode_of(dev, steps: int):
    """The two selection modes the paper uses on their own (end of Section III-B), on the language-model and image
    shapes: pure data selection (k = n, Eq. 12-20) and pure expert selection (c = m, Eq. 21-26), each timed through
    its shortcut and through the general routed path (UOE_FLAG_GENERAL_PATH), whole block forward, same protocol
    as the small workloads (L2 flushed before every step, one CUDA event pair per step)."""
    import torch

    import paper_2503_02495_b200 as uoe
    from paper_2503_02495_b200.workload import problem_of, to_dev

    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    out = {}
    for name in ("cfg2_lm", "cfg4_vit"):
        w0 = gen.WORKLOADS[name]
        for mode, w in (("data_selection_k=n", w0.replace(k=w0.n)), ("expert_selection_c=m", w0.replace(c=w0.m))):
            h = host_inputs(w)
            wd = {k: to_dev(v, dev) for k, v in h.items() if k not in ("x", "dy")}
            x_dev = to_dev(h["x"], dev)
            rec = {"k": w.k, "n": w.n, "c": w.c, "m": w.m, "routed_rows": w.R}
            ys = []
            for label, general in (("shortcut_ms", False), ("general_path_ms", True)):
                pa, pm = problem_of(w, "att", general_path=general), problem_of(w, "mlp", general_path=general)
                ws = uoe.alloc_block_workspace(pa, pm, dev)
                u, y = torch.empty_like(x_dev), torch.empty_like(x_dev)
                run = lambda: uoe.uoe_block_forward(pa, pm, x_dev, wd, u=u, y=y, ws=ws, check=False)
                for _ in range(3):
                    run()
                torch.cuda.synchronize()
                ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
                for e0, e1 in ev:
                    flush.zero_()
                    e0.record(stream)
                    run()
                    e1.record(stream)
                torch.cuda.synchronize()
                st = uoe.uoe_read_device_status(ws)
                if st != 0:
                    raise RuntimeError("device status in the single-mode run: " + uoe.status_string(st))
                rec[label] = sum(e0.elapsed_time(e1) for e0, e1 in ev) / steps
                ys.append(y.clone())
            rec["saved_us"] = (rec["general_path_ms"] - rec["shortcut_ms"]) * 1e3
            rec["same_bits"] = bool(torch.equal(ys[0], ys[1]))
            out[name + ":" + mode] = rec
    del flush
    torch.cuda.empty_cache()
    return out


TENSOR_KERNELS = ("gemm1_act", "gemm2", "mlp_fused", "qkv_proj", "out_proj", "attention", "bwd_da_dh", "bwd_dx", "wgrad_W1", "wgrad_W2",
                  "attn_bwd_dkdv", "attn_bwd_dq", "bwd_do", "bwd_dx_att", "wgrad_Wo", "wgrad_Wqkv")
HBM_KERNELS = ("route", "gather", "combine", "pool")


# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu captures summarised under profiles/.  Every
# entry names the source file of its kernel and that file's SHA-1 at the time of the capture: when the file has
# changed since, the line reports null instead of a stale figure.  (workload, kernel label) ->
# (bytes per launch at the benchmark's size, source file, sha1 prefix, profiles/ summary)
NCU_TRAFFIC = {
    ("cfg5_scale", "wgrad_W2"): (942.9e6, "wgrad_tcgen05.cu", "60af6e835bc7", "profiles/dram_traffic_per_kernel.md"),
    ("cfg5_scale", "wgrad_W1"): (862.4e6, "wgrad_tcgen05.cu", "60af6e835bc7", "profiles/dram_traffic_per_kernel.md"),
    ("cfg5_scale", "gemm1_act"): (943.1e6, "gemm_tcgen05.cu", "e9e4cad6259f", "profiles/dram_traffic_per_kernel.md"),
    ("cfg5_scale", "gemm2"): (951.1e6, "gemm2_patch_tcgen05.cu", "873f38bdafbd", "profiles/dram_traffic_per_kernel.md"),
    ("cfg5_scale", "bwd_da_dh"): (1106.9e6, "gemm_tcgen05.cu", "e9e4cad6259f", "profiles/dram_traffic_per_kernel.md"),
    ("cfg5_scale", "bwd_dx"): (934.7e6, "gemm2_patch_tcgen05.cu", "873f38bdafbd", "profiles/dram_traffic_per_kernel.md"),
    ("cfg5_scale", "route"): (271.9e6, "route.cu", "b4b9b9429eca", "profiles/dram_traffic_per_kernel.md"),
    ("cfg2_lm", "route"): (8.5e6, "route.cu", "b4b9b9429eca", "profiles/dram_traffic_per_kernel.md"),
    ("cfg2_lm", "mlp_fused"): (12.3e6, "mlp_fused_tcgen05.cu", "dbfbf455fb44", "profiles/dram_traffic_per_kernel.md"),
    ("cfg2_lm", "attention"): (6.9e6, "attn_tcgen05.cu", "4e097eabc901", "profiles/dram_traffic_per_kernel.md"),
    ("cfg2_lm", "combine"): (25.2e6, "routed.cu", "a26f173c1050", "profiles/dram_traffic_per_kernel.md"),
    ("cfg2_lm", "qkv_proj"): (9.7e6, "gemm_tcgen05.cu", "e9e4cad6259f", "profiles/dram_traffic_per_kernel.md"),
    ("cfg3_long", "route"): (16.9e6, "route.cu", "b4b9b9429eca", "profiles/dram_traffic_per_kernel.md"),
    ("cfg3_long", "mlp_fused"): (9.0e6, "mlp_fused_tcgen05.cu", "dbfbf455fb44", "profiles/dram_traffic_per_kernel.md"),
    ("cfg3_long", "attention"): (6.5e6, "attn_tcgen05.cu", "4e097eabc901", "profiles/dram_traffic_per_kernel.md"),
    ("cfg3_long", "combine"): (25.2e6, "routed.cu", "a26f173c1050", "profiles/dram_traffic_per_kernel.md"),
    ("cfg3_long", "qkv_proj"): (8.3e6, "gemm_tcgen05.cu", "e9e4cad6259f", "profiles/dram_traffic_per_kernel.md"),
    ("cfg4_vit", "route"): (38.8e6, "route.cu", "b4b9b9429eca", "profiles/dram_traffic_per_kernel.md"),
    ("cfg4_vit", "mlp_fused"): (55.7e6, "mlp_fused_tcgen05.cu", "dbfbf455fb44", "profiles/dram_traffic_per_kernel.md"),
    ("cfg4_vit", "attention"): (39.5e6, "attn_tcgen05.cu", "4e097eabc901", "profiles/dram_traffic_per_kernel.md"),
    ("cfg4_vit", "combine"): (123.7e6, "routed.cu", "a26f173c1050", "profiles/dram_traffic_per_kernel.md"),
    ("cfg4_vit", "qkv_proj"): (39.9e6, "gemm_tcgen05.cu", "e9e4cad6259f", "profiles/dram_traffic_per_kernel.md"),
}


def traffic_of(workload: str, kernel: str):
    ent = NCU_TRAFFIC.get((workload, kernel))
    if ent is None:
        return None
    import hashlib
    nbytes, src, sha, _summary = ent
    try:
        cur = hashlib.sha1(open(os.path.join(ROOT, "paper_2503_02495_b200", "csrc", src), "rb").read()).hexdigest()
    except OSError:
        return None
    return nbytes if cur.startswith(sha) else None


def roofline_of(top, w: gen.Workload, peaks, peak_src, sustained: bool = False):
    wk = work_table(w).get(top["kernel"], dict(flops=0, bytes=0))
    tpeak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    t_tensor = wk["flops"] / (tpeak * 1e12)
    t_hbm = wk["bytes"] / (peaks["hbm_gbs"] * 1e9)
    if t_tensor >= t_hbm and wk["flops"] > 0:
        roof = {"bound": "tensor", "achieved": top["tflops"], "peak": tpeak, "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": top["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": traffic_of(w.name, top["kernel"]),
                 "kernel": top["kernel"],
                 "avg_ms": top["avg_ms"], "share_of_kernel_time": top["share"],
                 "peak_source": peak_src + (" (sustained figure)" if sustained else " (burst figure)"),
                 "algorithmic_flops": wk["flops"], "algorithmic_bytes": wk["bytes"]})
    return roof


def block_of(w: gen.Workload, m, peaks, peak_src, world: int, ms_step: float, e2e_ms, args):
    """Everything reported for one workload, from one measure_gpu result."""
    flops = step_flops(w)
    kern = m["kernels"]
    k_by = {r["kernel"]: r for r in kern}
    tens = [k_by[n] for n in TENSOR_KERNELS if n in k_by]
    wt = work_table(w)
    tf_sum = sum(wt[r["kernel"]]["flops"] for r in tens)
    tm_sum = sum(r["avg_ms"] * r["launches_per_step"] for r in tens)
    blk = {
        "config": config_of(w, world, m["l2"]),
        "steps": args.steps, "ms_per_step": ms_step, "ms_per_step_min": m["ms_min"],
        "tokens_per_s": job_throughput(w, world, ms_step),
        "routed_rows_per_s": w.R * world / (ms_step * 1e-3),
        "tflops": flops * world / (ms_step * 1e-3) / 1e12,
        "frac_of_bf16_peak": flops / (ms_step * 1e-3) / 1e12 / peaks["bf16_tflops"],
        "algorithmic_gflop_per_step": flops / 1e9,
        "gpu_launches": m["launches"], "clocks": m["clocks"],
        "roofline": roofline_of(kern[0], w, peaks, peak_src),
        "tensor_kernels": {"tflops": tf_sum / tm_sum / 1e9, "frac_of_bf16_peak": tf_sum / tm_sum / 1e9 / peaks["bf16_tflops"]}
                          if tm_sum > 0 and w.dtype == "bf16" else None,
        "hbm_kernels": {n: {"gbs": k_by[n]["gbs"], "frac_of_hbm_peak": k_by[n]["gbs"] / peaks["hbm_gbs"]}
                        for n in HBM_KERNELS if n in k_by and n != "route"},
        "kernels": [{kk: (round(vv, 5) if isinstance(vv, float) else vv) for kk, vv in r.items()} for r in kern],
    }
    if "route_call" in m:
        rc = m["route_call"]
        blk["hbm_kernels"]["uoe_route (whole call)"] = {"ms": rc["ms"], "gbs": rc["gbs"], "frac_of_hbm_peak": rc["gbs"] / peaks["hbm_gbs"],
                                                         "timing": "CUDA events around %d calls in a stream" % rc["calls"],
                                                         "kernels": rc["kernels"], "sum_of_kernel_event_pairs_ms": rc["kernels_ms"]}
    if e2e_ms is not None:
        blk["e2e"] = {"value": w.B * w.L_valid * world / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
                      "steps": m.get("e2e_steps"), "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"]}
    if "sustained" in m:
        s = m["sustained"]
        tf = flops / (s["ms_per_step"] * 1e-3) / 1e12
        blk["sustained"] = {"steps": s["steps"], "seconds": s["seconds"], "ms_per_step": s["ms_per_step"],
                            "tokens_per_s": w.B * w.L_valid / (s["ms_per_step"] * 1e-3), "tflops": tf,
                            "frac_of_bf16_sustained_peak": tf / peaks["bf16_tflops_sustained"],
                            "frac_of_bf16_burst_peak": tf / peaks["bf16_tflops"], "clocks": s["clocks"]}
    if "parity" in m:
        blk["parity"] = m["parity"]
    return blk


def run_ours(args, w: gen.Workload, rank: int, local_rank: int, world: int):
    import torch
    import torch.distributed as dist

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    solo = world == 1 and args.part == "all"
    m = measure_gpu(args, w, dev, world, args.steps, args.warmup, True, with_parity=solo and not args.skip_cpu_baseline,
                    sustain_s=1.2 if solo and not args.no_sustained else 0.0)
    ms_step, e2e_ms = max_over_ranks([m["ms_step"], m["e2e_ms"]], world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks, peak_src = load_peaks()
    top = block_of(w, m, peaks, peak_src, world, ms_step, e2e_ms, args)
    if not args.skip_cpu_baseline:
        top["cpu_baseline"] = cpu_baseline_of(w, m["host"])
    del m

    line = base_line(w, args, world, top["config"]["l2"])
    line.update({"value": top["tokens_per_s"], "ms_per_step": ms_step, "ms_per_step_min": top["ms_per_step_min"],
                 "tflops": top["tflops"], "frac_of_bf16_peak": top["frac_of_bf16_peak"],
                 "e2e": top["e2e"], "gpu_launches": top["gpu_launches"], "clocks": top["clocks"],
                 "roofline": top["roofline"],
                 "cpu_baseline": top.get("cpu_baseline", {"value": None, "unit": "tokens/s", "cores": blas_threads(),
                                                          "kind": "oracle", "sample": "skipped"})})
    for key in ("sustained", "parity", "tensor_kernels", "hbm_kernels", "kernels", "routed_rows_per_s", "algorithmic_gflop_per_step"):
        if key in top:
            line[key] = top[key]

    # ---- the other workloads (language-model, long-sequence, image and the small float32 shapes), same protocol ----
    if solo and not args.no_others and args.B == 0 and not args.backward:
        others = {}
        for name in ALL_WORKLOADS:
            if name == w.name:
                continue
            wo = gen.WORKLOADS[name]
            mo = measure_gpu(args, wo, dev, 1, args.steps, args.warmup, True, with_parity=not args.skip_cpu_baseline,
                             sustain_s=1.2)
            bo = block_of(wo, mo, peaks, peak_src, 1, mo["ms_step"], mo["e2e_ms"], args)
            if not args.skip_cpu_baseline:
                bo["cpu_baseline"] = cpu_baseline_of(wo, mo["host"], budget_s=4.0)
            del mo
            others[name] = bo
        line["workloads"] = others
        line["single_mode"] = single_mode_of(dev, min(args.steps, 50))
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=TOP_WORKLOAD, choices=sorted(gen.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--B", type=int, default=0, help="override the workload's batch size (profiling on a smaller case)")
    ap.add_argument("--skip-cpu-baseline", action="store_true", help="omit the oracle timing and the parity block (profiling runs)")
    ap.add_argument("--backward", action="store_true", help="add the backward of every half of the block to the step")
    ap.add_argument("--part", default="all", choices=["all", "route"], help="time only a part of the step (profiling runs)")
    ap.add_argument("--no-sustained", action="store_true", help="omit the second-long sustained run (profiling runs)")
    ap.add_argument("--no-others", "--no-scale", dest="no_others", action="store_true",
                    help="only the selected workload: do not add the other workloads' blocks to the line")
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
