#!/usr/bin/env python
"""Benchmark of the truncated spectral layer (forward partial DFT, channel mixing,
inverse partial DFT, backward) on synthetic 3D+time FNO-shaped data.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one batch: F, M, I, then B.
Prints ONE JSON line (rank 0).  `value` is whole-job grid points per second for
fwd+bwd with inputs resident in HBM; `e2e` is the same through host buffers;
`roofline` is the dominant kernel against the measured HBM copy bandwidth;
`cpu_baseline` is the float64 oracle timed on this host on a bounded sample.
With --impl reference the oracle itself is the timed arm.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "spectral_layer_fwd_bwd_grid_points_per_s"
UNIT = "Gpoints/s"
DEFAULT_WORKLOAD = "cfg5_4d_128"
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            d = json.load(fh)
        return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, plain copy)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock, power and throttle reasons while the timed region runs (read-only NVML queries from a
    thread, every 10 ms: a child nvidia-smi takes longer to start than a short timed region lasts)."""

    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"),
               (0x4, "sw_power_cap"))

    def __init__(self, gpu_index: int, uuid=None):
        self.gpu = gpu_index
        self.uuid = uuid
        self.thread = None
        self.samples = []
        self.stop_flag = False
        self.nvml = None
        self.handle = None

    def _open(self):
        import pynvml
        pynvml.nvmlInit()
        self.nvml = pynvml
        handle = None
        if self.uuid:
            for cand in (f"GPU-{self.uuid}", str(self.uuid)):
                try:
                    handle = pynvml.nvmlDeviceGetHandleByUUID(cand)
                    break
                except Exception:
                    handle = None
        if handle is None:
            visible = os.environ.get("CUDA_VISIBLE_DEVICES", "")
            idx = self.gpu
            parts = [t for t in visible.split(",") if t.strip()]
            if parts and self.gpu < len(parts) and parts[self.gpu].strip().isdigit():
                idx = int(parts[self.gpu])
            handle = pynvml.nvmlDeviceGetHandleByIndex(idx)
        self.handle = handle
        self.max_sm = pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM)

    def _sample(self):
        n, h = self.nvml, self.handle
        sm = n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM)
        try:
            power = n.nvmlDeviceGetPowerUsage(h) / 1000.0
        except Exception:
            power = None
        try:
            getter = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                n.nvmlDeviceGetCurrentClocksThrottleReasons
            mask = int(getter(h))
        except Exception:
            mask = 0
        self.samples.append((sm, power, mask))

    def _run(self):
        import time as _t
        while not self.stop_flag:
            try:
                self._sample()
            except Exception:
                break
            _t.sleep(0.01)

    def start(self):
        try:
            self._open()
            self._sample()
            import threading
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()
        except Exception:
            self.thread = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.nvml is None or self.handle is None:
            return out
        try:
            self._sample()
        except Exception:
            pass
        self.stop_flag = True
        if self.thread is not None:
            self.thread.join(timeout=2)
        if self.samples:
            sm = [t[0] for t in self.samples]
            power = [t[1] for t in self.samples if t[1] is not None]
            mask = 0
            for t in self.samples:
                mask |= t[2]
            out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": self.max_sm,
                   "reasons": sorted(name for bit, name in self.REASONS if mask & bit),
                   "samples": len(sm), "power_w_max": max(power) if power else None}
        try:
            self.nvml.nvmlShutdown()
        except Exception:
            pass
        return out


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the two grid-streaming kernels from ncu
# captures of the same kernels at the same shape with FEWER CHANNELS (the capture-size rule: a few GB on the device
# at most under a multi-pass capture).  Two captures (2 and 4 channels) give a line: the slope is the traffic per
# channel, the intercept what does not grow with the tensor (a store stream's last dirty lines are still in L2 when
# the kernel ends and are counted by nobody), so the full launch is intercept + slope * channels instead of a
# plain scaling of one capture.  The summaries with their command lines are under profiles/.
NCU_TRAFFIC = {
    "cfg5_4d_128": {
        "channels": (2, 4),
        "grid_read": (1087604500, 2178791168),      # read + write bytes per launch at 2 and at 4 channels
        "grid_write": (1080980500, 2218048512),
        "source": "profiles/plane_kernels_cfg5_shape_c2_c4_ncu.md",
    },
}


def measured_traffic(workload: str, kind: str, channels: int):
    """Extrapolated DRAM traffic of one launch at `channels` channels, or None without a capture."""
    rec = NCU_TRAFFIC.get(workload)
    if not rec or kind not in rec:
        return None
    (c0, c1), (t0, t1) = rec["channels"], rec[kind]
    if t0 is None:
        return None
    if t1 is None:                       # one capture only: plain scaling (under-counts the fixed L2 residue)
        return t0 * channels / c0
    slope = (t1 - t0) / (c1 - c0)
    return t0 + slope * (channels - c0)


def algorithmic_bytes(w):
    """Bytes the method must move (grid read/written once, W streamed, spectra in and out)."""
    pts = w.B * w.points
    grid_in, grid_out = 4 * w.C_in * pts, 4 * w.C_out * pts
    Wb = 8 * w.C_in * w.C_out * w.M
    Xb, Yb = 8 * w.B * w.C_in * w.M, 8 * w.B * w.C_out * w.M
    fwd = grid_in + grid_out + Wb + 2 * Xb + 2 * Yb
    bwd = grid_out + grid_in + 2 * Wb + 2 * Yb + 2 * Xb + Xb
    return {"fwd": fwd, "fwd_bwd": fwd + bwd, "grid_read_launch_F": grid_in + Xb,
            "grid_read_launch_B": grid_out + Yb, "grid_write_launch_I": grid_out + Yb,
            "grid_write_launch_B": grid_in + Xb, "mix": Wb + Xb + Yb, "mix_adjoint": 2 * Wb + 2 * Xb + 2 * Yb}


# ----------------------------------------------------------------------------- the oracle as a timed arm
def oracle_sample_spec(w, budget=1.7e7):
    """A bounded sample of the workload for the CPU oracle: a slab of planes along dim 0
    (with its global phase offset, Eq. 18) and a subset of channels, sized for a few seconds."""
    work = w.B * w.points * max(w.C_in, w.C_out)
    # budget = point-channels per step (1.7e7 is about a second of oracle work on 8 cores)
    cs = 1 if work > budget else min(w.C_in, w.C_out)
    n0 = w.N[0]
    while n0 > 1 and w.B * (w.points // w.N[0]) * n0 * cs > budget and n0 % 2 == 0:
        n0 //= 2
    return cs, n0


def run_oracle_step(w, cs, n0, data):
    from oracle import dtst_oracle as O
    x, W, g = data
    off = (0,) * w.d
    nl_N = w.N
    if n0 != w.N[0]:
        kw = dict(N_global=w.N, offsets=off)
    else:
        kw = {}
    y, Xhat = O.layer_forward(x, W, w.kmax, **kw)
    gx, gW = O.backward(g, Xhat, W.reshape((cs, cs) + w.K), w.kmax, **kw)
    return float(y.ravel()[0] + gx.ravel()[0])


def oracle_data(w, cs, n0):
    import numpy as np
    from paper_2607_14394_b200 import inputs
    x = np.stack([np.stack([inputs.make_field_channel(w, b, c)[:n0] for c in range(cs)]) for b in range(w.B)])
    g = np.stack([np.stack([inputs.make_upstream_grad_channel(w, b, c)[:n0] for c in range(cs)]) for b in range(w.B)])
    W = inputs.make_weights(w, cs, cs)
    return x, W, g


ORACLE_BUDGET = 1.7e7      # point-channels per sample step: about a second of oracle work on 8 cores


def time_oracle(w, steps, warmup, budget=ORACLE_BUDGET, one_core=True):
    """Times the oracle as it stands on a bounded sample of the workload: `warmup` untimed steps (at least one),
    then `steps` timed ones, mean and min; then the same on ONE core (threadpoolctl) when asked."""
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threadpool_limits = None
        threads = len(os.sched_getaffinity(0))
    cs, n0 = oracle_sample_spec(w, budget)
    data = oracle_data(w, cs, n0)

    def run(n_warm, n_steps):
        for _ in range(n_warm):
            run_oracle_step(w, cs, n0, data)
        ts = []
        for _ in range(n_steps):
            t0 = time.perf_counter()
            run_oracle_step(w, cs, n0, data)
            ts.append(time.perf_counter() - t0)
        return sum(ts) / len(ts), min(ts)

    dt, dt_min = run(max(1, warmup), max(1, steps))
    sample_ptch = w.B * (w.points // w.N[0]) * n0 * cs
    # equivalent whole-layer grid points per second at the workload's channel count
    to_value = lambda t: sample_ptch / max(w.C_in, w.C_out) / t / 1e9
    value = to_value(dt)
    grid_part = (f"the whole grid" if n0 == w.N[0] else
                 f"first {n0} of {w.N[0]} planes along dim 0 (a slab, with its global phase offset)")
    sample = (f"float64 numpy oracle, fwd+bwd, {cs} of {w.C_in} channels (in and out), {grid_part}; "
              f"value = sample point-channels / {max(w.C_in, w.C_out)} channels / time; "
              f"{max(1, warmup)} warm-up + {max(1, steps)} timed sample steps, mean (min also given)")
    info = {"kind": "oracle", "cores": int(min(threads, len(os.sched_getaffinity(0)))),
            "host_cores": len(os.sched_getaffinity(0)), "sample": sample,
            "seconds_per_sample_step": dt, "seconds_per_sample_step_min": dt_min, "value_at_min": to_value(dt_min)}
    if one_core and threadpool_limits is not None:
        try:
            with threadpool_limits(limits=1):
                dt1, dt1_min = run(0, max(1, min(steps, 2)))
            info["one_core"] = {"value": to_value(dt1), "unit": UNIT, "cores": 1, "seconds_per_sample_step": dt1,
                                "seconds_per_sample_step_min": dt1_min}
        except Exception as ex:
            info["one_core"] = {"error": f"{type(ex).__name__}: {ex}"[:120]}
    return value, dt, info


def main_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    steps, warmup = max(1, args.steps), max(1, args.warmup)
    value, dt, info = time_oracle(w, steps, warmup)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "C_in": w.C_in, "C_out": w.C_out, "grid": list(w.N),
                   "kmax": list(w.kmax), "note": "the CPU oracle on a bounded sample; ms_per_step is per sample step"},
        "cpu_baseline": dict(info, value=value, unit=UNIT),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------- our arm
def torch_fft_reference(torch, w, x, W, g, steps=3):
    """Secondary reference point on the same GPU: rfftn -> slice -> einsum -> zero-pad -> irfftn (fp32)."""
    out = {}
    try:
        d = w.d
        dims = tuple(range(2, 2 + d))
        idx = []
        for j in range(d):
            k, n = w.kmax[j], w.N[j]
            idx.append(torch.cat([torch.arange(k), torch.arange(n - k, n)]).cuda() if j < d - 1 else torch.arange(k).cuda())
        ix = torch.meshgrid(*idx, indexing="ij")
        Wm = W.reshape((w.C_in, w.C_out) + w.K)
        letters = "xyzt"[:d]

        def fwd(xx, WW):
            Xf = torch.fft.rfftn(xx, dim=dims)
            Xs = Xf[(slice(None), slice(None)) + tuple(ix)]
            del Xf
            Ys = torch.einsum(f"bi{letters},io{letters}->bo{letters}", Xs, WW)
            full = torch.zeros((w.B, w.C_out) + tuple(w.N[:-1]) + (w.N[-1] // 2 + 1,), dtype=torch.complex64,
                               device=xx.device)
            full[(slice(None), slice(None)) + tuple(ix)] = Ys
            return torch.fft.irfftn(full, s=w.N, dim=dims)

        with torch.no_grad():
            fwd(x, Wm)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                y = fwd(x, Wm)
            e1.record()
            torch.cuda.synchronize()
            del y
        t = e0.elapsed_time(e1) / steps
        out["fwd_ms"] = t
        out["fwd_gpoints_per_s"] = w.B * w.points / (t * 1e-3) / 1e9
        try:
            xr = x.detach().clone().requires_grad_(True)
            Wr = Wm.detach().clone().requires_grad_(True)
            for it in range(steps + 1):
                if it == 1:
                    torch.cuda.synchronize()
                    e0.record()
                xr.grad = None
                Wr.grad = None
                y = fwd(xr, Wr)
                y.backward(g)
                del y
            e1.record()
            torch.cuda.synchronize()
            t2 = e0.elapsed_time(e1) / steps
            out["fwd_bwd_ms"] = t2
            out["fwd_bwd_gpoints_per_s"] = w.B * w.points / (t2 * 1e-3) / 1e9
        except Exception as ex:  # typically out of memory at the largest grids
            out["fwd_bwd_error"] = type(ex).__name__
        out["what"] = "torch.fft.rfftn -> slice -> einsum -> zero-pad -> irfftn, fp32, same GPU"
    except Exception as ex:
        out["error"] = f"{type(ex).__name__}: {ex}"[:200]
    finally:
        torch.cuda.empty_cache()
    return out


def graph_step_ms(torch, step_fn, steps=10):
    """One step captured in a CUDA graph (the compute calls allocate nothing and never synchronise, so they can be
    captured as they are) and replayed: the step time without per-launch host overhead."""
    try:
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.stream(side):
            step_fn()
            torch.cuda.synchronize()
            with torch.cuda.graph(graph, stream=side):
                step_fn()
        torch.cuda.synchronize()
        for _ in range(3):
            graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        del graph
        return ms
    except Exception as ex:
        return f"{type(ex).__name__}: {ex}"[:160]


def timed_steps(torch, plan, tensors, steps, barrier=None, sampler=None, instrument=False):
    """`steps` whole steps (F, M, I, B) between two synchronisations, timed with CUDA events on the launching
    stream around the region.  With `instrument` the region also carries an event after every phase and the
    library's own events around the dominant kernels (per-phase and per-kernel times); an event between two
    kernels keeps the second from starting its prologue under the first one's tail (programmatic dependent
    launch), so the headline step time is taken WITHOUT them and the instrumented pass follows it."""
    x, g, W, Xhat, Yhat, y, gx, gW = tensors

    def step(evs=None):
        if evs is not None:
            evs[0].record()
        plan.forward(x, Xhat)
        if evs is not None:
            evs[1].record()
        plan.spectral_mul(Xhat, W, Yhat)
        if evs is not None:
            evs[2].record()
        plan.inverse(Yhat, y)
        if evs is not None:
            evs[3].record()
        plan.backward(g, Xhat, W, gx, gW)
        if evs is not None:
            evs[4].record()

    if instrument:
        plan.enable_kernel_timing(2 * steps + 2)
    phase_events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] if instrument else None
                    for _ in range(steps)]
    launches0 = plan.launch_count()
    if barrier:
        barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(steps):
        step(phase_events[i])
    t_end.record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    clocks = sampler.stop() if sampler else None
    launches = plan.launch_count() - launches0
    ms_step = t_start.elapsed_time(t_end) / steps
    out = {"ms_step": ms_step, "launches": launches, "clocks": clocks, "step_fn": step}
    if instrument:
        out["phases"] = [sum(phase_events[i][j].elapsed_time(phase_events[i][j + 1]) for i in range(steps)) / steps
                         for j in range(4)]
        out["kt"] = {k: plan.kernel_timing(k) for k in ("grid_read", "grid_write", "mix", "mix_adjoint")}
        plan.enable_kernel_timing(0)
    return out


def kernel_table(w, kt):
    """Per kernel kind: launches, average launch time, algorithmic bytes per launch and the rate they give."""
    ab = algorithmic_bytes(w)

    def kind_line(kind, bytes_per_launch):
        n, ms = kt[kind]
        if n == 0:
            return None
        avg = ms / n
        return {"launches": n, "avg_ms": avg, "algorithmic_bytes_per_launch": bytes_per_launch,
                "achieved_gbs": bytes_per_launch / (avg * 1e-3) / 1e9}

    return {
        "grid_read": kind_line("grid_read", (ab["grid_read_launch_F"] + ab["grid_read_launch_B"]) / 2),
        "grid_write": kind_line("grid_write", (ab["grid_write_launch_I"] + ab["grid_write_launch_B"]) / 2),
        "mix": kind_line("mix", ab["mix"]),
        "mix_adjoint": kind_line("mix_adjoint", ab["mix_adjoint"]),
    }


def virtual_shard_summary(torch, w, x, g, W, P, steps, peak):
    """The headline workload once more with its dimension 0 cut into P virtual slabs (partial spectra with global
    phase offsets, summed on the device in ascending order), timed exactly like the headline: same number of
    steps, phase split, kernel table, whole-step roofline fraction."""
    from paper_2607_14394_b200 import Plan
    try:
        plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P)
        X = plan.forward(x)
        Y = plan.spectral_mul(X, W)
        y = plan.inverse(Y)
        gx, gW = plan.backward(g, X, W)
        tensors = (x, g, W, X, Y, y, gx, gW)
        for _ in range(3):
            plan.forward(x, X)
            plan.spectral_mul(X, W, Y)
            plan.inverse(Y, y)
            plan.backward(g, X, W, gx, gW)
        torch.cuda.synchronize()
        ms = timed_steps(torch, plan, tensors, steps)["ms_step"]
        r = timed_steps(torch, plan, tensors, steps, instrument=True)
        ok = plan.status() == 0
        ab = algorithmic_bytes(w)
        out = {"P": P, "ms_per_step": ms, "ms_per_step_instrumented": r["ms_step"], "gpoints_per_s": w.B * w.points / ms / 1e6, "status_ok": ok, "steps": steps,
               "phases_ms": dict(zip("FMIB", r["phases"])), "kernels": kernel_table(w, r["kt"]),
               "gpu_launches": r["launches"],
               "algorithmic_gbs": ab["fwd_bwd"] / (ms * 1e-3) / 1e9,
               "frac_of_measured_peak": ab["fwd_bwd"] / (ms * 1e-3) / 1e9 / peak,
               "frac_of_nominal_8TBs": ab["fwd_bwd"] / (ms * 1e-3) / 1e9 / 8000.0}
        plan.close()
        del plan, X, Y, y, gx, gW, tensors, r
        torch.cuda.empty_cache()
        return out
    except Exception as ex:
        return {"P": P, "error": f"{type(ex).__name__}: {ex}"[:200]}


def block_summary(torch, w, x, g, W, steps, peak):
    """The whole block of Algorithm 1 on the headline workload - GELU(W_bypass x + layer(x)) with the pre-activation
    kept for training, and its backward pass - timed like the headline (K uninstrumented steps, then K with the
    library's events around the block's own kernels).  Algorithmic bytes: the layer's, plus one more read of x for
    the bypass, plus (training) the pre-activation written once and read once, g_z written and read once, x and
    grad_x read once more for the bypass adjoint."""
    from paper_2607_14394_b200 import Plan
    try:
        dev = x.device
        plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
        gen = torch.Generator(device=dev).manual_seed(w.seed + 77)
        Wb = torch.randn((w.C_out, w.C_in), device=dev, generator=gen) / w.C_in ** 0.5
        out, Xhat, z = plan.block_forward(x, W, Wb)
        scratch = torch.empty_like(z)
        gx, gW, gWb = plan.block_backward(g, x, z, Xhat, W, Wb, scratch=scratch)

        def fwd():
            plan.block_forward(x, W, Wb, out, Xhat, z)

        def bwd():
            plan.block_backward(g, x, z, Xhat, W, Wb, scratch, gx, gW, gWb)

        for _ in range(3):
            fwd()
            bwd()
        torch.cuda.synchronize()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record()
        for _ in range(steps):
            fwd()
        e[1].record()
        for _ in range(steps):
            bwd()
        e[2].record()
        torch.cuda.synchronize()
        tf, tb = e[0].elapsed_time(e[1]) / steps, e[1].elapsed_time(e[2]) / steps
        plan.enable_kernel_timing(steps + 2)
        for _ in range(steps):
            fwd()
            bwd()
        torch.cuda.synchronize()
        kt = {k: plan.kernel_timing(k) for k in ("block_epilogue", "gelu_backward", "bypass_backward")}
        # the forward epilogue once more with each of its two kernels asked for explicitly
        epi = {}
        for mode in ("ffma", "tensor"):
            try:
                plan.set_block_epilogue(mode)
                fwd()
                torch.cuda.synchronize()
                plan.kernel_timing("block_epilogue")
                for _ in range(steps):
                    fwd()
                n_e, ms_e = plan.kernel_timing("block_epilogue")
                epi[mode] = ms_e / max(1, n_e)
            except Exception as ex:
                epi[mode] = f"{type(ex).__name__}"[:60]
        plan.set_block_epilogue("auto")
        plan.enable_kernel_timing(0)
        ok = plan.status() == 0
        ab = algorithmic_bytes(w)
        pts = w.B * w.points
        gin, gout = 4 * w.C_in * pts, 4 * w.C_out * pts
        bytes_f = ab["fwd"] + gin + 2 * gout                  # x once more; z written; y/out read-modify-written
        bytes_b = (ab["fwd_bwd"] - ab["fwd"]) + 3 * gout + gout + gin + 2 * gin   # gelu' pass, bypass adjoint pass
        kernel_bytes = {"block_epilogue": gin + 3 * gout, "gelu_backward": 3 * gout, "bypass_backward": gout + 3 * gin}
        res = {"fwd_ms": tf, "fwd_bwd_ms": tf + tb, "status_ok": ok, "steps": steps,
               "fwd_gpoints_per_s": pts / tf / 1e6, "fwd_bwd_gpoints_per_s": pts / (tf + tb) / 1e6,
               "bytes_moved_model": {"fwd": bytes_f, "fwd_bwd": bytes_f + bytes_b},
               "fwd_gbs": bytes_f / tf / 1e6, "fwd_bwd_gbs": (bytes_f + bytes_b) / (tf + tb) / 1e6,
               "fwd_bwd_frac_of_measured_peak": (bytes_f + bytes_b) / (tf + tb) / 1e6 / peak,
               "bypass_product": "auto: fp32 FFMA with the input channels in registers (the faster kernel at every "
                                 "channel count measured); tcgen05.mma kind::tf32 (3xTF32, accumulator in TMEM) on request",
               "epilogue_kernel_ms": {"ffma": epi.get("ffma"), "tcgen05": epi.get("tensor")},
               "kernels": {k: {"launches": n, "avg_ms": ms / n, "bytes_per_launch": kernel_bytes[k],
                               "achieved_gbs": kernel_bytes[k] / (ms / n) / 1e6,
                               "frac_of_measured_peak": kernel_bytes[k] / (ms / n) / 1e6 / peak}
                           for k, (n, ms) in kt.items() if n}}
        plan.close()
        del plan, out, Xhat, z, scratch, gx, gW, gWb
        torch.cuda.empty_cache()
        return res
    except Exception as ex:
        return {"error": f"{type(ex).__name__}: {ex}"[:200]}


def fno_summary(torch, steps=5):
    """A whole synthetic FNO with the paper's architecture (Section "Experimental Setup": 4 Fourier blocks, modes
    (8, 8, 8, 16), 5 fields in and out, grid 128 x 128 x 64 with a time axis of 32 or 30) forward and backward on
    this GPU, every step in the library's kernels: at the paper's width 20 and at width 32 (the channel counts the
    tensor-core bypass kernels serve).  Random-init weights, synthetic input; context for the paper's multi-GPU
    figures, not a like-for-like comparison."""
    from paper_2607_14394_b200 import FNO
    out = {"grid": [128, 128, 64, "time_axis"], "modes": [8, 8, 8, 16], "layers": 4, "fields": 5, "steps": steps,
           "paper_context": "the paper reports 148.3 ms forward / 246.8 ms backward for this architecture at "
                            "128^3 on 4 V100s (its Table 5); another machine, another grid: context only"}
    # (time axis, width, key): the paper's operation count is on a time axis of 30 points, which runs on the row
    # kernels for any extent; 32 points run on the plane kernels
    for T, width, key in ((32, 20, "width_20"), (32, 32, "width_32"), (30, 20, "t30_width_20")):
        try:
            net = FNO((128, 128, 64, T), (8, 8, 8, 16), 1, 5, 5, width, 4, seed=11)
            gen = torch.Generator(device="cuda").manual_seed(12)
            a = torch.randn((1, 5, 128, 128, 64, T), device="cuda", generator=gen)
            gu = torch.randn((1, 5, 128, 128, 64, T), device="cuda", generator=gen)
            for _ in range(2):
                net.forward(a)
                net.backward(gu)
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            fwd = bwd = 0.0
            for _ in range(steps):
                e[0].record()
                net.forward(a)
                e[1].record()
                net.backward(gu)
                e[2].record()
                torch.cuda.synchronize()
                fwd += e[0].elapsed_time(e[1])
                bwd += e[1].elapsed_time(e[2])
            ok = net.plan.status() == 0
            out[key] = {"fwd_ms": fwd / steps, "bwd_ms": bwd / steps, "status_ok": ok,
                        "kernel_path": net.plan.kernel_path, "time_axis": T}
            net.close()
            del net, a, gu
            torch.cuda.empty_cache()
        except Exception as ex:
            out[key] = {"error": f"{type(ex).__name__}: {ex}"[:200]}
    return out


def other_configs_summary(torch, skip_name, steps=10):
    """Forward and forward+backward time of the other benchmark configurations (parity-test cases, not the
    headline) and of the paper's own layer on both of its time axes: seeded device-generated inputs of each shape,
    CUDA events, 3 warm-ups."""
    from paper_2607_14394_b200 import Plan, inputs
    out = {}
    cases = [(name, w, "tf32x3") for name, w in list(inputs.WORKLOADS.items()) + list(inputs.EXTRA_WORKLOADS.items())]
    # the paper's layer once more with single-pass TF32 products (a plan option with a stated error of 2e-3)
    cases.append(("paper_4d_t30_tf32", inputs.EXTRA_WORKLOADS["paper_4d_t30"], "tf32"))
    for name, w, arithmetic in cases:
        if name == skip_name:
            continue
        try:
            dev = torch.device("cuda", torch.cuda.current_device())
            plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, arithmetic=arithmetic)
            gen = torch.Generator(device=dev)
            gen.manual_seed(w.seed)
            x = torch.randn((w.B, w.C_in) + w.N, device=dev, generator=gen)
            g = torch.randn((w.B, w.C_out) + w.N, device=dev, generator=gen)
            W = inputs.make_weights_torch(w, dev)
            X = plan.forward(x)
            Y = plan.spectral_mul(X, W)
            y = plan.inverse(Y)
            gx, gW = plan.backward(g, X, W)

            def fwd():
                plan.forward(x, X)
                plan.spectral_mul(X, W, Y)
                plan.inverse(Y, y)

            for _ in range(3):
                fwd()
                plan.backward(g, X, W, gx, gW)
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
            for _ in range(steps):
                fwd()
            e[1].record()
            for _ in range(steps):
                plan.backward(g, X, W, gx, gW)
            e[2].record()
            torch.cuda.synchronize()
            tf, tb = e[0].elapsed_time(e[1]) / steps, e[1].elapsed_time(e[2]) / steps

            def whole_step():
                fwd()
                plan.backward(g, X, W, gx, gW)

            tg = graph_step_ms(torch, whole_step, steps)
            ab = algorithmic_bytes(w)
            pts = w.B * w.points
            out[name] = {"kernel_path": plan.kernel_path, "arithmetic": arithmetic, "fwd_ms": tf, "fwd_bwd_ms": tf + tb,
                         "fwd_gpoints_per_s": pts / tf / 1e6, "fwd_bwd_gpoints_per_s": pts / (tf + tb) / 1e6,
                         "fwd_algorithmic_gbs": ab["fwd"] / tf / 1e6,
                         "fwd_bwd_algorithmic_gbs": ab["fwd_bwd"] / (tf + tb) / 1e6,
                         "fwd_bwd_cuda_graph_ms": tg,
                         "grid_bytes": 4 * w.C_in * pts,
                         "note": "grid smaller than L2: warm-cache, launch-bound" if 4 * w.C_in * pts < 126e6 else
                                 "grid larger than L2"}
            plan.close()
            del plan, x, g, W, X, Y, y, gx, gW
            torch.cuda.empty_cache()
        except Exception as ex:
            out[name] = {"error": f"{type(ex).__name__}: {ex}"[:160]}
    return out


def main_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2607_14394_b200 import Plan, inputs
    from paper_2607_14394_b200 import dist as D

    world, rank, local_rank = D.env_world()
    if world > 1 and args.multi == "slab":
        return main_sharded(args, w)
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the spectral layer has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    D.init_process_group("nccl", dev)

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    P = args.shards
    # --channels is a profiler aid that runs the full workload's kernels on fewer tasks: keep the kernel choice of
    # the full workload (with few channels the automatic choice would drop the fused third dimension)
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P, path=args.path,
                column_contraction=1 if args.channels else 0)

    # the batch each rank works on is its own (weak scaling over independent samples; no collective)
    x = inputs.make_field_torch(w, dev, tag=0, rank=rank)
    g = inputs.make_field_torch(w, dev, tag=1, rank=rank)
    W = inputs.make_weights_torch(w, dev, rank=0)
    Xhat = torch.empty((w.B, w.C_in) + w.K, dtype=torch.complex64, device=dev)
    Yhat = torch.empty((w.B, w.C_out) + w.K, dtype=torch.complex64, device=dev)
    y = torch.empty((w.B, w.C_out) + w.N, dtype=torch.float32, device=dev)
    gx = torch.empty((w.B, w.C_in) + w.N, dtype=torch.float32, device=dev)
    gW = torch.empty((w.C_in, w.C_out, w.M), dtype=torch.complex64, device=dev)
    tensors = (x, g, W, Xhat, Yhat, y, gx, gW)

    def barrier():
        if world > 1:
            dist.barrier()

    def warm_fwd():
        plan.forward(x, Xhat)
        plan.spectral_mul(Xhat, W, Yhat)
        plan.inverse(Yhat, y)

    def warm():
        warm_fwd()
        plan.backward(g, Xhat, W, gx, gW)

    for _ in range(warmup):
        warm()
    torch.cuda.synchronize()
    if plan.status() != 0:
        raise RuntimeError("device-side status word set during warm-up")

    sampler = ClockSampler(local_rank, uuid=getattr(torch.cuda.get_device_properties(local_rank), "uuid", None)) \
        if rank == 0 else None
    r0 = timed_steps(torch, plan, tensors, steps, barrier, sampler)
    clocks, launches, ms_step, step = r0["clocks"], r0["launches"], r0["ms_step"], r0["step_fn"]
    # second pass of the same K steps with events after every phase and around the dominant kernels
    r = timed_steps(torch, plan, tensors, steps, barrier, None, instrument=True)
    ph, kt, ms_instr = r["phases"], r["kt"], r["ms_step"]
    # and the forward half alone (F, M, I), uninstrumented like the headline
    barrier()
    torch.cuda.synchronize()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record()
    for _ in range(steps):
        warm_fwd()
    f1.record()
    torch.cuda.synchronize()
    fwd_only_ms = f0.elapsed_time(f1) / steps
    graph_ms = graph_step_ms(torch, step, min(steps, 10)) if (rank == 0 and world == 1 and
                                                             not args.no_other_configs) else None

    red = D.max_over_ranks([ms_step, ms_instr, fwd_only_ms] + ph, device=dev)
    ms_step, ms_instr, fwd_only_ms, ph = red[0], red[1], red[2], red[3:]

    pts_per_step = world * w.B * w.points
    value = D.whole_job_throughput(w.B * w.points, ms_step, world) / 1e9
    fwd_ms = fwd_only_ms
    ab = algorithmic_bytes(w)
    peak, peak_src = measured_peaks()

    # roofline of the dominant kernel kind (the two grid-streaming kernels carry ~all bytes)
    kinds = kernel_table(w, kt)
    dom = max((k for k in ("grid_read", "grid_write") if kinds[k]), key=lambda k: kt[k][1], default=None)
    roofline = None
    if dom:
        a = kinds[dom]["achieved_gbs"]
        traffic = measured_traffic(w.name.split("_c")[0] if args.channels else w.name, dom, w.C_in)
        roofline = {"bound": "hbm", "kernel": dom, "achieved": a, "peak": peak, "unit": "GB/s", "frac": a / peak,
                    "frac_of_nominal_8TBs": a / 8000.0, "traffic": traffic,
                    "traffic_over_algorithmic": (traffic / kinds[dom]["algorithmic_bytes_per_launch"]) if traffic else None,
                    "peak_source": peak_src, "avg_launch_ms": kinds[dom]["avg_ms"]}
    # the whole step against the same roof: every algorithmic byte of F, M, I, B over the step time
    step_gbs = ab["fwd_bwd"] / (ms_step * 1e-3) / 1e9
    roofline_step = {"bound": "hbm", "algorithmic_bytes": ab["fwd_bwd"], "achieved": step_gbs, "peak": peak,
                     "unit": "GB/s", "frac": step_gbs / peak, "frac_of_nominal_8TBs": step_gbs / 8000.0,
                     "peak_source": peak_src, "target_frac_of_nominal": 0.70,
                     "fwd": {"algorithmic_bytes": ab["fwd"], "achieved": ab["fwd"] / (fwd_ms * 1e-3) / 1e9,
                             "frac": ab["fwd"] / (fwd_ms * 1e-3) / 1e9 / peak,
                             "frac_of_nominal_8TBs": ab["fwd"] / (fwd_ms * 1e-3) / 1e9 / 8000.0}}

    # end to end through host buffers: pinned host -> device copies of x and g_y, the step,
    # device -> host reads of y, grad_x and grad_W, all inside the timed region
    e2e = None
    if args.no_e2e:
        e2e = {"value": None, "unit": UNIT, "skipped": "--no-e2e"}
    elif rank == 0 or world > 1:
        # Every rank pins five host buffers (43 GB at this workload); all ranks of the node must get theirs, and
        # they decide TOGETHER whether to run, so that no rank waits at a barrier for one that gave up.
        hx = hg = hy = hgx = hgW = None
        pinned_ok = 1.0
        try:
            need = 4 * (x.numel() + g.numel() + y.numel() + gx.numel()) + 8 * gW.numel()
            try:
                import psutil
                if need * world > 0.7 * psutil.virtual_memory().available:
                    pinned_ok = 0.0
            except ImportError:
                pass
            if pinned_ok:
                hx = torch.empty(x.shape, dtype=torch.float32, pin_memory=True)
                hg = torch.empty(g.shape, dtype=torch.float32, pin_memory=True)
                hy = torch.empty(y.shape, dtype=torch.float32, pin_memory=True)
                hgx = torch.empty(gx.shape, dtype=torch.float32, pin_memory=True)
                hgW = torch.empty(gW.shape, dtype=torch.complex64, pin_memory=True)
        except Exception:
            pinned_ok = 0.0
        if world > 1:
            flag = torch.tensor([pinned_ok], device=dev)
            dist.all_reduce(flag, op=dist.ReduceOp.MIN)
            pinned_ok = float(flag.item())
        if not pinned_ok:
            hx = hg = hy = hgx = hgW = None
            e2e = {"value": None, "unit": UNIT, "skipped": "pinned host buffers for every rank did not fit host memory"}
    if e2e is None and (rank == 0 or world > 1):
        try:
            e2e_steps = max(1, min(steps, args.e2e_steps))
            from paper_2607_14394_b200.binding import HostPipeline
            hx.copy_(x)
            hg.copy_(g)
            del x, g, y, gx, gW, tensors, r, r0, step
            torch.cuda.empty_cache()
            pipe = HostPipeline(plan, W)
            pipe.step(hx, hg, hy, hgx, hgW)            # warm-up
            pipe.wait()
            torch.cuda.synchronize()
            barrier()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            a0.record()                                # idle device: the event completes at once
            for _ in range(e2e_steps):
                pipe.step(hx, hg, hy, hgx, hgW)
            pipe.wait()                                # the library's own wait: every output is in host memory
            a1.record()
            torch.cuda.synchronize()
            ms_host = (time.perf_counter() - t0) * 1e3 / e2e_steps
            ms_e = a0.elapsed_time(a1) / e2e_steps
            barrier()
            ms_e = D.max_over_ranks([ms_e], device=dev)[0]
            y_check = float(hy.view(-1)[:1024].double().abs().sum())
            e2e = {"value": pts_per_step / (ms_e * 1e-3) / 1e9, "unit": UNIT,
                   "h2d_bytes_per_step": int(hx.numel() * 4 + hg.numel() * 4),
                   "d2h_bytes_per_step": int(hy.numel() * 4 + hgx.numel() * 4 + hgW.numel() * 8),
                   "ms_per_step": ms_e, "ms_per_step_host_clock": ms_host, "steps": e2e_steps,
                   "result_checksum": y_check,
                   "what": "pinned host x, grad_y -> device; F, M, I, B; y, grad_x, grad_W -> pinned host; copies "
                           "overlap compute on the library's three internal streams (dtst_step_host through the "
                           "C ABI with host pointers); CUDA events on an idle device before the first call and "
                           "after dtst_host_io_wait returned"}
            pipe.close()
            del pipe
            torch.cuda.empty_cache()
            x, g = hx.to(dev), hg.to(dev)
            del hx, hg, hy, hgx, hgW
        except Exception as ex:
            e2e = {"value": None, "unit": UNIT, "error": f"{type(ex).__name__}: {ex}"[:200]}

    line = None
    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "ms_per_step_instrumented": ms_instr,
            "config": {"workload": w.name, "B_per_gpu": w.B, "C_in": w.C_in, "C_out": w.C_out, "grid": list(w.N),
                       "kmax": list(w.kmax), "modes": w.M, "field": w.field, "virtual_shards": P,
                       "kernel_path": plan.kernel_path, "l2": "inputs larger than L2 (no flush needed)"
                       if 4 * w.B * w.C_in * w.points > 3 * 126e6 else "inputs smaller than L2: warm-cache numbers",
                       "parallelism": f"independent batches x{world}, no collective",
                       "launches_per_step": launches // max(1, steps),
                       "forward_third_dimension": "contracted inside the plane kernel" if launches // max(1, steps) <= 12
                       and plan.kernel_path == "fused" and w.d >= 3 and P == 1 and w.name == "cfg5_4d_128"
                       else "separate launch or not applicable"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches,
            "roofline": roofline, "roofline_step": roofline_step,
            "fwd": {"ms": fwd_ms, "gpoints_per_s": pts_per_step / (fwd_ms * 1e-3) / 1e9,
                    "algorithmic_gbs": ab["fwd"] / (fwd_ms * 1e-3) / 1e9,
                    "frac_of_measured_peak": ab["fwd"] / (fwd_ms * 1e-3) / 1e9 / peak},
            "fwd_bwd": {"ms": ms_step, "gpoints_per_s": value, "point_channels_per_s_G": value * w.C_in,
                        "algorithmic_gbs": ab["fwd_bwd"] / (ms_step * 1e-3) / 1e9,
                        "frac_of_measured_peak": ab["fwd_bwd"] / (ms_step * 1e-3) / 1e9 / peak,
                        "frac_of_nominal_8TBs": ab["fwd_bwd"] / (ms_step * 1e-3) / 1e9 / 8000.0},
            "phases_ms": {"F": ph[0], "M": ph[1], "I": ph[2], "B": ph[3],
                          "note": "from the instrumented pass (an event after every phase)"},
            "kernels": kinds,
            "paper_context": "paper reports 38-64x forward / 37x training speedup of DRIFT over a distributed FNO "
                             "on 4-32 V100s (multi-node communication); not comparable to a single-GPU number",
        }
    # secondary reference and CPU baseline: rank 0, single GPU only
    if rank == 0 and world == 1:
        torch.cuda.empty_cache()
        if graph_ms is not None:
            line["cuda_graph"] = {"ms_per_step": graph_ms,
                                  "what": "the same step captured once in a CUDA graph and replayed"}
        if not args.no_other_configs and args.channels == 0 and P == 1 and w.virtual_shards > 1:
            line["virtual_shards"] = virtual_shard_summary(torch, w, x, g, W, w.virtual_shards, steps, peak)
        if not args.no_other_configs:
            line["block"] = block_summary(torch, w, x, g, W, min(steps, 10), peak)
        if not args.no_torch_ref:
            line["torch_fft_reference"] = torch_fft_reference(torch, w, x, W, g)
        if not args.no_other_configs and args.channels == 0:
            del x, g
            torch.cuda.empty_cache()
            line["other_configs"] = other_configs_summary(torch, w.name)
            line["fno"] = fno_summary(torch)
        if not args.no_cpu_baseline:
            try:
                # the same bounded sample, warm-up and statistics as the reference arm (--impl reference)
                v, dt, info = time_oracle(w, args.cpu_steps, 1)
                line["cpu_baseline"] = dict(info, value=v, unit=UNIT)
            except Exception as ex:
                line["cpu_baseline"] = {"value": None, "unit": UNIT, "kind": "oracle", "cores": 0,
                                        "sample": f"failed: {type(ex).__name__}: {ex}"[:200]}
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main_sharded(args, w):
    """N > 1 ranks, one per GPU: the layer sharded the way Algorithm 1 shards it (strong scaling).  The workload's
    grid is cut into N slabs along dimension 0 and its modes and weights into N equal chunks; per step every rank
    runs forward and backward with two collectives per direction (all-reduce of the partial spectrum, all-gather
    of the mixed chunks), the received spectra landing in local memory before any kernel reads them.  Timed with
    CUDA events between barriers, max over ranks; rank 0 prints the JSON line.

    `--backend gloo --ops-module MODULE:FACTORY` runs the same launcher and the same exchange logic on CPU ranks
    with a stand-in for the CUDA steps supplied by the caller (the tests do that); such a line is marked
    "data_path": "stand-in" and is not a measurement of this library."""
    import torch
    import torch.distributed as dist
    from paper_2607_14394_b200 import dist as D
    from paper_2607_14394_b200 import inputs
    from paper_2607_14394_b200.dist_layer import SlabShardedLayer

    world, rank, local_rank = D.env_world()
    gloo = args.backend == "gloo"
    if gloo:
        if not args.ops_module:
            raise RuntimeError("--backend gloo needs --ops-module: the layer itself has no CPU path")
        import importlib
        mod, fn = args.ops_module.split(":")
        make_ops = getattr(importlib.import_module(mod), fn)
        dev = torch.device("cpu")
        D.init_process_group("gloo")
    else:
        if not torch.cuda.is_available():
            raise RuntimeError("bench.py needs CUDA devices: the spectral layer has no CPU path")
        if local_rank >= torch.cuda.device_count():
            raise RuntimeError(f"rank {rank} has no GPU: {torch.cuda.device_count()} visible, {world} ranks")
        dev = torch.device("cuda", local_rank)
        torch.cuda.set_device(dev)
        D.init_process_group("nccl", dev)
    if w.N[0] % world != 0 or w.M % world != 0:
        raise RuntimeError(f"{world} ranks must divide N_0 = {w.N[0]} and the mode count {w.M}")
    n_local = (w.N[0] // world,) + tuple(w.N[1:])
    offset = (rank * n_local[0],) + (0,) * (w.d - 1)
    ops = make_ops(w.N, n_local, offset, w.kmax, w.B, w.C_in, w.C_out) if gloo else None
    layer = SlabShardedLayer(w.N, w.kmax, w.B, w.C_in, w.C_out, world, rank, device=dev, ops=ops)

    steps, warmup = max(1, args.steps), max(3, args.warmup)
    gen = torch.Generator(device=dev)
    gen.manual_seed(D.rank_seed(w.seed, rank))
    rdt = torch.float64 if gloo else torch.float32
    cdt = torch.complex128 if gloo else torch.complex64
    x = torch.randn((w.B, w.C_in) + n_local, generator=gen, device=dev, dtype=rdt)
    g = torch.randn((w.B, w.C_out) + n_local, generator=gen, device=dev, dtype=rdt)
    W_shard = torch.view_as_complex(torch.randn((w.C_in, w.C_out, layer.cnt, 2), generator=gen, device=dev, dtype=rdt)
                                    / (w.C_in * w.C_out) ** 0.5).to(cdt)

    class Clock:
        """CUDA events on the launching stream, or the host clock for the CPU stand-in."""
        def __init__(self):
            self.t = torch.cuda.Event(enable_timing=True) if not gloo else None
        def record(self):
            if gloo:
                self.t = time.perf_counter()
            else:
                self.t.record()
        def ms_to(self, other):
            return (other.t - self.t) * 1e3 if gloo else self.t.elapsed_time(other.t)

    PH = ("F_local", "all_reduce_X", "mix", "all_gather_Y", "I_local",
          "B_spectrum_local", "all_reduce_GY", "mix_adjoint", "all_gather_GX", "B_input_local")

    def step(marks=None):
        def m(i):
            if marks is not None:
                marks[i].record()
        m(0)
        Xp = layer.local_spectrum(x); m(1)
        Xhat = layer._all_reduce(Xp, None); m(2)
        Yc = layer.local_mix(Xhat, W_shard); m(3)
        Yhat = layer._all_gather(Yc, None); m(4)
        y = layer.local_inverse(Yhat); m(5)
        GYp = layer.local_grad_spectrum(g); m(6)
        GY = layer._all_reduce(GYp, None); m(7)
        GXc, gWs = layer.local_grad_mix(GY, Xhat, W_shard); m(8)
        GX = layer._all_gather(GXc, None); m(9)
        gx = layer.local_grad_input(GX); m(10)
        return y, gx, gWs

    def sync():
        if not gloo:
            torch.cuda.synchronize()

    for _ in range(warmup if not gloo else 1):
        step()
    sync()
    if not gloo and layer.ops.plan.status() != 0:
        raise RuntimeError("device-side status word set during warm-up")
    launches0 = 0 if gloo else layer.ops.plan.launch_count()
    sampler = None
    if rank == 0 and not gloo:
        sampler = ClockSampler(local_rank, uuid=getattr(torch.cuda.get_device_properties(local_rank), "uuid", None))
    marks = [[Clock() for _ in range(11)] for _ in range(steps)]
    dist.barrier()
    sync()
    if sampler:
        sampler.start()
    for i in range(steps):
        step(marks[i])
    sync()
    dist.barrier()
    clocks = sampler.stop() if sampler else None
    ms_step = marks[0][0].ms_to(marks[-1][10]) / steps
    ph = [sum(marks[i][j].ms_to(marks[i][j + 1]) for i in range(steps)) / steps for j in range(10)]
    red = D.max_over_ranks([ms_step] + ph, device=dev)
    ms_step, ph = red[0], red[1:]
    launches = 0 if gloo else layer.ops.plan.launch_count() - launches0

    # end to end: every step copies this rank's slab of x and grad_y from pinned host memory and reads y, grad_x
    # and the grad_W shard back (plain stream-ordered copies around the same step)
    e2e = None
    if not gloo and not args.no_e2e:
        try:
            hx, hg = x.cpu().pin_memory(), g.cpu().pin_memory()
            hy, hgx = torch.empty_like(hx).pin_memory() if w.C_in == w.C_out else \
                torch.empty((w.B, w.C_out) + n_local).pin_memory(), torch.empty_like(hx).pin_memory()
            hgW = torch.empty((w.C_in, w.C_out, layer.cnt), dtype=torch.complex64).pin_memory()

            def e2e_step():
                x.copy_(hx, non_blocking=True)
                g.copy_(hg, non_blocking=True)
                y, gx, gWs = step()
                hy.copy_(y, non_blocking=True)
                hgx.copy_(gx, non_blocking=True)
                hgW.copy_(gWs, non_blocking=True)

            e2e_step()
            sync()
            dist.barrier()
            n_e = max(1, min(steps, args.e2e_steps))
            a0, a1 = Clock(), Clock()
            a0.record()
            for _ in range(n_e):
                e2e_step()
            a1.record()
            sync()
            dist.barrier()
            ms_e = D.max_over_ranks([a0.ms_to(a1) / n_e], device=dev)[0]
            e2e = {"value": w.B * w.points / (ms_e * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": ms_e, "steps": n_e,
                   "h2d_bytes_per_step": int(world * 4 * (hx.numel() + hg.numel())),
                   "d2h_bytes_per_step": int(world * (4 * (hy.numel() + hgx.numel()) + 8 * hgW.numel())),
                   "what": "every rank: its slab of x, grad_y pinned host -> device; the sharded step; its slab of "
                           "y, grad_x and its grad_W shard -> pinned host; bytes are the job's total"}
        except Exception as ex:
            e2e = {"value": None, "unit": UNIT, "error": f"{type(ex).__name__}: {ex}"[:200]}
    elif not gloo:
        e2e = {"value": None, "unit": UNIT, "skipped": "--no-e2e"}

    if rank == 0:
        pts = w.B * w.points                       # the GLOBAL grid: total work is fixed as N grows
        ab = algorithmic_bytes(w)
        peak, peak_src = measured_peaks()
        spectrum_bytes = 8 * w.B * w.M
        line = {
            "metric": METRIC, "value": pts / (ms_step * 1e-3) / 1e9, "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup if not gloo else 1, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f64" if gloo else "f32", "data": "synthetic",
            "config": {"workload": w.name, "B": w.B, "C_in": w.C_in, "C_out": w.C_out, "grid": list(w.N),
                       "kmax": list(w.kmax), "modes": w.M, "slab_per_rank": list(n_local),
                       "modes_per_rank": layer.cnt, "l2": "inputs larger than L2 (no flush needed)"
                       if 4 * w.B * w.C_in * w.points / world > 3 * 126e6 else "per-rank inputs smaller than L2",
                       "parallelism": f"slab{world} along dim 0: all-reduce of the partial spectrum, mode-sharded "
                                      f"mixing, all-gather (per direction); backend {args.backend}"},
            "backend": args.backend, "data_path": "stand-in (test ops on CPU ranks)" if gloo else "cuda",
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches) * world,
            "phases_ms": dict(zip(PH, ph)),
            "collective_ms_per_step": ph[1] + ph[3] + ph[6] + ph[8],
            "collective_payload_bytes_per_step": {
                "all_reduce": spectrum_bytes * (w.C_in + w.C_out),
                "all_gather": spectrum_bytes * (w.C_out + w.C_in)},
            "roofline_step": None if gloo else {
                "bound": "hbm", "algorithmic_bytes": ab["fwd_bwd"],
                "achieved": ab["fwd_bwd"] / (ms_step * 1e-3) / 1e9, "peak": peak * world, "unit": "GB/s",
                "frac": ab["fwd_bwd"] / (ms_step * 1e-3) / 1e9 / (peak * world), "peak_source": peak_src + f" x {world}"},
        }
        print(json.dumps(line))
    dist.destroy_process_group()
    return 0


def respawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` without a launcher: start N ranks of this very script under torchrun (one per
    GPU, rendezvous on 127.0.0.1) and hand their output through."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=DEFAULT_WORKLOAD)
    ap.add_argument("--shards", type=int, default=1, help="virtual shards along dim 0")
    ap.add_argument("--path", default="auto", choices=["auto", "generic"])
    ap.add_argument("--e2e-steps", type=int, default=6)
    ap.add_argument("--channels", type=int, default=0,
                    help="override C_in = C_out (smaller cases for profiler captures; not a bench configuration)")
    ap.add_argument("--multi", default="slab", choices=["slab", "batches"],
                    help="N > 1: 'slab' = the layer sharded over ranks (Algorithm 1, strong scaling, collectives); "
                         "'batches' = an independent batch per rank (weak scaling, no collective)")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"])
    ap.add_argument("--ops-module", default="", help="with --backend gloo: MODULE:FACTORY of a stand-in for the CUDA steps")
    ap.add_argument("--cpu-steps", type=int, default=3, help="timed sample steps of the CPU oracle baseline")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-torch-ref", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true")
    args = ap.parse_args()
    from paper_2607_14394_b200 import inputs
    w = inputs.workload(args.config)
    if args.channels > 0:
        w = inputs.custom_workload(f"{w.name}_c{args.channels}", w.B, args.channels, args.channels, w.N, w.kmax,
                                   field=w.field, seed=w.seed, virtual_shards=w.virtual_shards)
    if args.impl == "reference":
        return main_reference(args, w)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return respawn_ranks(args.gpus)
    return main_ours(args, w)


if __name__ == "__main__":
    sys.exit(main())
