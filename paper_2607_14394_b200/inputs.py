"""Seeded synthetic inputs for the truncated spectral layer.

This module only draws random numbers and shapes them; it contains none of the
method's arithmetic (no partial DFT, no mode selection, no channel mixing).  It
is the single piece shared by the CPU oracle's callers and the CUDA path's
callers, so that both sides see identical bits.

The workloads stand in for the paper's 3D+time FNO inputs (Section "Dataset":
PDEBench 3D compressible Navier-Stokes trajectories initialised from random
fields), which are not available here: smooth fields are Gaussian random fields
with an isotropic power spectrum proportional to |k|^-2.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One configuration of the spectral layer (shapes only)."""

    name: str
    B: int
    C_in: int
    C_out: int
    N: tuple          # grid extents, last one contiguous (the rfft dimension)
    kmax: tuple       # retained modes per dimension
    field: str        # "iid" | "grf" | "grf+noise"
    seed: int
    virtual_shards: int = 1

    @property
    def d(self) -> int:
        return len(self.N)

    @property
    def K(self) -> tuple:
        """Retained entries per dimension: 2k on the two-sided dims, k on the last."""
        return tuple(2 * k for k in self.kmax[:-1]) + (self.kmax[-1],)

    @property
    def M(self) -> int:
        return math.prod(self.K)

    @property
    def points(self) -> int:
        return math.prod(self.N)


# The five configurations of the benchmark definition, in its order.
WORKLOADS = {
    "cfg1_2d_64": Workload("cfg1_2d_64", 1, 4, 4, (64, 64), (8, 8), "iid", 1001),
    "cfg2_3d_64": Workload("cfg2_3d_64", 2, 16, 16, (64, 64, 64), (12, 12, 12), "grf+noise", 1002),
    "cfg3_4d_64": Workload("cfg3_4d_64", 1, 8, 8, (64, 64, 64, 32), (8, 8, 8, 4), "grf", 1003),
    "cfg4_3d_256": Workload("cfg4_3d_256", 1, 32, 32, (256, 256, 256), (16, 16, 16), "iid", 1004),
    "cfg5_4d_128": Workload("cfg5_4d_128", 1, 16, 16, (128, 128, 128, 64), (16, 16, 16, 8), "grf", 1005,
                            virtual_shards=8),
}

# The paper's own layer (Section "Experimental Setup": grid 128 x 128 x 64, modes (8, 8, 8, 16), width 20), with the
# time axis of its operation count (30 points: no multiple of 32, every one-sided mode retained) and with 32 points.
# Not part of the benchmark definition: bench.py takes them by name, the tests do not iterate over them.
EXTRA_WORKLOADS = {
    "paper_4d_t30": Workload("paper_4d_t30", 1, 20, 20, (128, 128, 64, 30), (8, 8, 8, 16), "grf", 1006),
    "paper_4d_t32": Workload("paper_4d_t32", 1, 20, 20, (128, 128, 64, 32), (8, 8, 8, 16), "grf", 1007),
    # shapes of the usual 1-D and 2-D operator-learning problems (long rows, many batch entries, few modes): seeded
    # synthetic fields of these shapes, as everywhere
    "signal_1d_8192": Workload("signal_1d_8192", 20, 64, 64, (8192,), (16,), "grf", 1008),
    "grid_2d_1024": Workload("grid_2d_1024", 4, 32, 32, (1024, 1024), (12, 12), "grf", 1009),
    "grid_2d_421": Workload("grid_2d_421", 4, 32, 32, (421, 421), (12, 12), "grf", 1010),
}


def workload(name: str) -> Workload:
    return WORKLOADS[name] if name in WORKLOADS else EXTRA_WORKLOADS[name]


def _channel_rng(seed: int, tag: int, b: int, c: int) -> np.random.Generator:
    # One independent PCG64 stream per (tensor tag, batch, channel), so a single
    # channel of a large workload can be regenerated without the others.
    return np.random.default_rng([seed, tag, b, c])


def gaussian_random_field(rng: np.random.Generator, N: tuple, noise: float = 0.0) -> np.ndarray:
    """Real field on grid N with power spectrum ~ |k|^-2, unit sample variance.

    White complex Gaussian half-spectrum, amplitude |k|^-1 with signed integer
    wavenumbers, zero mean; an optional iid N(0, noise^2) term is added after
    normalisation.  Returned as float64.
    """
    d = len(N)
    half = tuple(N[:-1]) + (N[-1] // 2 + 1,)
    xi = rng.standard_normal(half) + 1j * rng.standard_normal(half)
    k2 = np.zeros(half, dtype=np.float64)
    for j in range(d):
        kj = np.fft.fftfreq(N[j]) * N[j] if j < d - 1 else np.arange(half[-1], dtype=np.float64)
        shape = [1] * d
        shape[j] = half[j]
        k2 = k2 + kj.reshape(shape) ** 2
    k2.flat[0] = 1.0
    amp = 1.0 / np.sqrt(k2)
    amp.flat[0] = 0.0
    f = np.fft.irfftn(xi * amp, s=N, axes=tuple(range(d)))
    f = f / f.std()
    if noise > 0.0:
        f = f + noise * rng.standard_normal(N)
    return f


def make_field_channel(w: Workload, b: int, c: int, tag: int = 0) -> np.ndarray:
    """One (b, c) channel of the input field as float32, shape N."""
    rng = _channel_rng(w.seed, tag, b, c)
    if w.field == "iid":
        f = rng.standard_normal(w.N)
    elif w.field == "grf":
        f = gaussian_random_field(rng, w.N)
    elif w.field == "grf+noise":
        f = gaussian_random_field(rng, w.N, noise=0.01)
    else:
        raise ValueError(w.field)
    return f.astype(np.float32)


def make_field(w: Workload, channels: int | None = None) -> np.ndarray:
    """x[B, C_in, *N] float32 (all channels; use make_field_channel for big grids)."""
    C = w.C_in if channels is None else channels
    out = np.empty((w.B, C) + tuple(w.N), dtype=np.float32)
    for b in range(w.B):
        for c in range(C):
            out[b, c] = make_field_channel(w, b, c, tag=0)
    return out


def make_upstream_grad_channel(w: Workload, b: int, c: int) -> np.ndarray:
    """One (b, o) channel of the upstream gradient g_y: iid N(0,1), float32."""
    return _channel_rng(w.seed, 1, b, c).standard_normal(w.N).astype(np.float32)


def make_upstream_grad(w: Workload, channels: int | None = None) -> np.ndarray:
    C = w.C_out if channels is None else channels
    out = np.empty((w.B, C) + tuple(w.N), dtype=np.float32)
    for b in range(w.B):
        for c in range(C):
            out[b, c] = make_upstream_grad_channel(w, b, c)
    return out


def make_weights(w: Workload, C_in: int | None = None, C_out: int | None = None) -> np.ndarray:
    """W[C_in, C_out, M] complex64; re and im iid N(0, var = 1/(C_in*C_out)).

    The variance always uses the workload's own channel counts, also when only
    a channel subset is requested.
    """
    ci = w.C_in if C_in is None else C_in
    co = w.C_out if C_out is None else C_out
    std = 1.0 / math.sqrt(w.C_in * w.C_out)
    out = np.empty((ci, co, w.M), dtype=np.complex64)
    for i in range(ci):
        rng = _channel_rng(w.seed, 2, i, 0)
        re = rng.standard_normal((w.C_out, w.M)) * std
        im = rng.standard_normal((w.C_out, w.M)) * std
        out[i] = (re[:co] + 1j * im[:co]).astype(np.complex64)
    return out


def make_spectrum(w: Workload, C: int, tag: int = 3) -> np.ndarray:
    """A random complex64 spectrum [B, C, M] (for testing the inverse alone)."""
    rng = _channel_rng(w.seed, tag, 0, 0)
    z = rng.standard_normal((w.B, C, w.M)) + 1j * rng.standard_normal((w.B, C, w.M))
    return z.astype(np.complex64)


def custom_workload(name, B, C_in, C_out, N, kmax, field="iid", seed=7, virtual_shards=1) -> Workload:
    return Workload(name, B, C_in, C_out, tuple(N), tuple(kmax), field, seed, virtual_shards)


# --------------------------------------------------------------------------
# Device-side generation for the large workloads (same recipe, torch RNG): a
# channel is produced directly in GPU memory; callers that need it on the host
# copy those very bits back, so both sides still see identical values.
# --------------------------------------------------------------------------
def make_field_channel_torch(w: Workload, b: int, c: int, device, tag: int = 0, rank: int = 0):
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(int(w.seed) * 1000003 + tag * 100003 + rank * 1009 + b * 131 + c)
    N = tuple(w.N)
    if w.field == "iid" or tag == 1:
        return torch.randn(N, device=device, dtype=torch.float32, generator=gen)
    d = len(N)
    half = N[:-1] + (N[-1] // 2 + 1,)
    xi = torch.randn(half + (2,), device=device, dtype=torch.float32, generator=gen)
    k2 = torch.zeros(half, device=device, dtype=torch.float32)
    for j in range(d):
        if j < d - 1:
            kj = torch.fft.fftfreq(N[j], device=device) * N[j]
        else:
            kj = torch.arange(half[-1], device=device, dtype=torch.float32)
        shape = [1] * d
        shape[j] = half[j]
        k2 = k2 + kj.reshape(shape) ** 2
    k2.view(-1)[0] = 1.0
    amp = torch.rsqrt(k2)
    amp.view(-1)[0] = 0.0
    spec = torch.view_as_complex(xi) * amp
    del xi, k2, amp
    f = torch.fft.irfftn(spec, s=N, dim=tuple(range(d)))
    del spec
    f = f / f.std()
    if w.field == "grf+noise":
        f = f + 0.01 * torch.randn(N, device=device, dtype=torch.float32, generator=gen)
    return f.contiguous()


def make_field_torch(w: Workload, device, tag: int = 0, channels: int | None = None, rank: int = 0):
    """x (tag 0, C_in channels) or the upstream gradient (tag 1, C_out channels, iid) on the device."""
    import torch

    C = channels if channels is not None else (w.C_in if tag == 0 else w.C_out)
    out = torch.empty((w.B, C) + tuple(w.N), device=device, dtype=torch.float32)
    for b in range(w.B):
        for c in range(C):
            out[b, c] = make_field_channel_torch(w, b, c, device, tag, rank)
    return out


def make_weights_torch(w: Workload, device, rank: int = 0):
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(int(w.seed) * 1000003 + 2 * 100003 + rank * 1009)
    std = 1.0 / math.sqrt(w.C_in * w.C_out)
    z = torch.randn((w.C_in, w.C_out, w.M, 2), device=device, dtype=torch.float32, generator=gen) * std
    return torch.view_as_complex(z).contiguous()
