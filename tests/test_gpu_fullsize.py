"""Parity at the benchmark's full sizes (the two large configurations), in the launch
configuration bench.py times.  The oracle cannot afford every channel of an 8.6 GB tensor,
so each output is checked on whole channels the oracle CAN compute (a channel of the layer's
grid-side stages is independent of the others), on single modes by the literal un-factored
sum of Eq. 5, and on sampled grid points by the literal sum of Eq. 14.  Inputs are seeded,
generated on the device, and the very same bits are copied to the host for the oracle."""
import math

import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import inputs as I
from parity_checks import per_mode_excess, per_plane_excess

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


def _lists(w):
    return O.mode_index_lists(w.N, w.kmax)


def _literal_points(Y_c, w, points, doubling=True, normalise=True):
    """y[n] at the given grid points for one channel, by the un-factored sum over all modes (Eq. 14)."""
    lists = _lists(w)
    c = O.hermitian_weights(w.N[-1], w.kmax[-1]) if doubling else np.ones(w.kmax[-1])
    out = []
    for n in points:
        ph = np.ones((), dtype=np.complex128)
        for j in range(w.d):
            r = np.mod(lists[j] * int(n[j]), w.N[j]).astype(np.float64)
            f = np.exp(2j * np.pi * r / w.N[j])
            shape = [1] * w.d
            shape[j] = len(lists[j])
            ph = ph * f.reshape(shape)
        v = np.sum(c * np.real(Y_c.astype(np.complex128) * ph))
        out.append(v / math.prod(w.N) if normalise else v)
    return np.array(out)


def _three_channels(C, rng):
    """The first and the last channel (lowest and highest row coordinates of the tensor) and a seeded random one."""
    mid = int(rng.integers(1, C - 1)) if C > 2 else 0
    return sorted({0, mid, C - 1})


def _check_layer_fullsize(w, P_list, rng_seed):
    from paper_2607_14394_b200 import Plan
    dev = torch.device("cuda")
    rng = np.random.default_rng(rng_seed)
    x = I.make_field_torch(w, dev, tag=0)
    W = I.make_weights_torch(w, dev)
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
    assert plan.kernel_path in ("fused", "row", "generic")
    lists = _lists(w)
    for j in range(w.d):
        assert plan.mode_indices(j) == lists[j].tolist()
    chans_in, chans_out = _three_channels(w.C_in, rng), _three_channels(w.C_out, rng)

    # ---- F: whole channels against the separable oracle (tensor norm and every mode on its own scale),
    # single modes against the literal sum
    Xhat = plan.forward(x)
    torch.cuda.synchronize()
    assert plan.status() == 0
    X_ref = {}
    c0 = chans_in[0]
    x_c0 = x[0, c0].cpu().numpy()
    for c in chans_in:
        X_ref[c] = O.forward(x[0, c].cpu().numpy()[None, None], w.kmax)[0, 0]
        got = Xhat[0, c].cpu().numpy()
        assert O.rel_l2(got, X_ref[c]) <= TOL, c
        assert per_mode_excess(got[None, None], X_ref[c][None, None]) <= 1.0, c
    for _ in range(3):
        pos = tuple(int(rng.integers(0, len(s))) for s in lists)
        v = O.forward_one_mode(x_c0, w.N, [lists[j][pos[j]] for j in range(w.d)])
        got = complex(Xhat[(0, c0) + pos].item())
        assert abs(got - v) <= 1e-5 * np.sqrt(np.mean(np.abs(X_ref[c0]) ** 2)) + 1e-5 * abs(v)
    del x_c0

    # ---- V: virtual shards against the unsharded device result and the oracle
    for P in P_list:
        planP = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P)
        XP = planP.forward(x)
        torch.cuda.synchronize()
        assert planP.status() == 0
        a = torch.view_as_real(XP).double()
        b = torch.view_as_real(Xhat).double()
        assert float((a - b).norm() / b.norm()) <= TOL
        for c in chans_in:
            assert O.rel_l2(XP[0, c].cpu().numpy(), X_ref[c]) <= TOL
            assert per_mode_excess(XP[0, c].cpu().numpy()[None, None], X_ref[c][None, None]) <= 1.0
        planP.close()
        del planP, XP, a, b
    del x
    torch.cuda.empty_cache()

    # ---- M: full size against the oracle's einsum, on an independent random spectrum
    Xs = torch.from_numpy(I.make_spectrum(w, w.C_in, tag=3).reshape((w.B, w.C_in) + w.K)).to(dev)
    Yhat = plan.spectral_mul(Xs, W)
    Y_ref = O.spectral_mul(Xs.cpu().numpy(), W.cpu().numpy().reshape((w.C_in, w.C_out) + w.K))
    assert O.rel_l2(Yhat.cpu().numpy(), Y_ref) <= TOL
    assert per_mode_excess(Yhat.cpu().numpy(), Y_ref) <= 1.0

    # ---- I: whole channels against the separable oracle (tensor norm and every plane), sampled points
    # against the literal sum
    y = plan.inverse(Yhat)
    torch.cuda.synchronize()
    for co in chans_out:
        y_ref = O.inverse(Y_ref[0, co][None, None], w.N, w.kmax)[0, 0]
        got = y[0, co].cpu().numpy()
        assert O.rel_l2(got, y_ref) <= TOL, co
        assert per_plane_excess(got[None, None], y_ref[None, None]) <= 1.0, co
    rms = float(np.sqrt(np.mean(y_ref ** 2)))
    cl = (chans_out[-1] + 1) % w.C_out
    pts = [tuple(int(rng.integers(0, n)) for n in w.N) for _ in range(24)]
    lit = _literal_points(Y_ref[0, cl], w, pts)
    got = np.array([float(y[(0, cl) + p].item()) for p in pts])
    assert np.max(np.abs(got - lit)) <= 2e-5 * rms
    del y_ref, got

    # ---- B: upstream gradient with three live channels (the others are exactly zero, which keeps the
    # oracle's share to three forward transforms while every kernel still runs at full size)
    live = chans_out
    g = torch.zeros((w.B, w.C_out) + w.N, device=dev)
    for o in live:
        g[0, o] = I.make_field_channel_torch(w, 0, o, dev, tag=1)
    gx, gW = plan.backward(g, Xs, W)
    torch.cuda.synchronize()
    assert plan.status() == 0
    cw = O.hermitian_weights(w.N[-1], w.kmax[-1])
    GY = {o: O.forward(g[0, o].cpu().numpy()[None, None], w.kmax)[0, 0] * cw / float(math.prod(w.N)) for o in live}
    Xs_h = Xs.cpu().numpy()
    W_h = W.cpu().numpy().reshape((w.C_in, w.C_out) + w.K)
    gW_h = gW.cpu().numpy().reshape((w.C_in, w.C_out) + w.K)
    for o in live:
        ref = np.conj(Xs_h[0]) * GY[o][None]               # [C_in, K...], B = 1
        assert O.rel_l2(gW_h[:, o], ref) <= TOL
        assert per_mode_excess(gW_h[:, o][None], ref[None]) <= 1.0
    dead = [o for o in range(w.C_out) if o not in live][0]
    assert float(np.abs(gW_h[:, dead]).max()) == 0.0
    gx_ref = {}
    for i0 in chans_in:
        GX = sum(GY[o] * np.conj(W_h[i0, o]) for o in live)
        gx_ref[i0] = O.inverse(GX[None, None], w.N, w.kmax, doubling=False, normalise=False)[0, 0]
        got = gx[0, i0].cpu().numpy()
        assert O.rel_l2(got, gx_ref[i0]) <= TOL, i0
        assert per_plane_excess(got[None, None], gx_ref[i0][None, None]) <= 1.0, i0

    # ---- I and B with virtual shards at full size: the expansions do not depend on the slabs (same kernels,
    # so the same bits); the backward's forward-type stage sums slab partials, so it matches within tolerance
    for P in P_list:
        planP = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P)
        yP = planP.inverse(Yhat)
        torch.cuda.synchronize()
        assert torch.equal(yP, y)
        del yP
        gxP, gWP = planP.backward(g, Xs, W)
        torch.cuda.synchronize()
        assert planP.status() == 0
        assert float((torch.view_as_real(gWP).double() - torch.view_as_real(gW).double()).norm() /
                     torch.view_as_real(gW).double().norm()) <= TOL
        i0 = chans_in[-1]
        got = gxP[0, i0].cpu().numpy()
        assert O.rel_l2(got, gx_ref[i0]) <= TOL
        assert per_plane_excess(got[None, None], gx_ref[i0][None, None]) <= 1.0
        for c in range(w.C_in):
            d = (gxP[0, c].double() - gx[0, c].double()).norm() / gx[0, c].double().norm()
            assert float(d) <= TOL, c
        planP.close()
        del planP, gxP, gWP
    plan.close()


def test_cfg5_4d_128_fullsize():
    w = I.WORKLOADS["cfg5_4d_128"]
    _check_layer_fullsize(w, P_list=[w.virtual_shards], rng_seed=55)


def test_cfg4_3d_256_fullsize():
    w = I.WORKLOADS["cfg4_3d_256"]
    _check_layer_fullsize(w, P_list=[4], rng_seed=44)


def test_paper_layer_time_axis_30_fullsize():
    """The paper's own layer at its width (20 channels, grid 128 x 128 x 64 x 30, modes (8, 8, 8, 16): Section
    "Experimental Setup" and the operation count of Section "cuBLAS vs cuFFT"), which runs on the kernels for
    contiguous extents that are no multiple of 32."""
    w = I.EXTRA_WORKLOADS["paper_4d_t30"]
    _check_layer_fullsize(w, P_list=[4], rng_seed=30)


def test_cfg5_shape_iid_field_every_mode_has_equal_weight():
    """The largest shape once more with a white field: every retained mode then has the same expected
    magnitude, so no mode's error can hide behind a stronger one (the smooth fields of the benchmark put
    most of their energy into the lowest modes)."""
    from paper_2607_14394_b200 import Plan
    w0 = I.WORKLOADS["cfg5_4d_128"]
    w = I.custom_workload("cfg5_iid", w0.B, 2, 2, w0.N, w0.kmax, field="iid", seed=2027)
    dev = torch.device("cuda")
    x = I.make_field_torch(w, dev, tag=0)
    for P in (1, w0.virtual_shards):
        plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P)
        assert plan.kernel_path == "fused"
        Xhat = plan.forward(x)
        torch.cuda.synchronize()
        assert plan.status() == 0
        for c in range(w.C_in):
            ref = O.forward(x[0, c].cpu().numpy()[None, None], w.kmax)
            got = Xhat[0, c].cpu().numpy()[None, None]
            assert O.rel_l2(got, ref) <= TOL
            assert per_mode_excess(got, ref) <= 1.0
            mags = np.abs(ref)
            assert mags.min() > 0.0 and np.median(mags) / np.sqrt(np.mean(mags ** 2)) > 0.5   # a flat spectrum
        plan.close()


@pytest.mark.parametrize("name", ["cfg5_4d_128", "cfg4_3d_256", "paper_4d_t30"])
def test_fullsize_properties_that_hold_at_any_size(name):
    """At the benchmark's full sizes, in its launch configuration, on every channel at once (no oracle needed):
    the adjoint identity <F x, Y> = <x, F^H Y> with F^H = dtst_backward_input, the pair
    <I Y, g> = <Y, G_Y(g)> with G_Y = dtst_backward_spectrum, and linearity of F."""
    from paper_2607_14394_b200 import Plan
    w = I.workload(name)
    dev = torch.device("cuda")
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
    gen = torch.Generator(device=dev).manual_seed(2024)
    x = torch.randn((w.B, w.C_in) + w.N, device=dev, generator=gen)
    Y = torch.randn((w.B, w.C_in) + w.K, dtype=torch.complex64, device=dev, generator=gen)

    def cdot(a, b):   # Re <a, b> over complex tensors, accumulated in float64
        return float((torch.view_as_real(a).double() * torch.view_as_real(b).double()).sum().item())

    def rdot(a, b):
        return float(torch.dot(a.reshape(-1).double(), b.reshape(-1).double()).item()) if a.numel() < 2 ** 31 else \
            float(sum(torch.dot(a[:, c].reshape(-1).double(), b[:, c].reshape(-1).double()).item()
                      for c in range(a.shape[1])))

    Fx = plan.forward(x)
    FhY = plan.backward_input(Y)                       # F^H Y on the grid (needs C_in channels)
    lhs, rhs = cdot(Fx, Y), rdot(x, FhY)
    assert abs(lhs - rhs) <= 2e-5 * max(abs(lhs), float(torch.view_as_real(Fx).double().norm() *
                                                      torch.view_as_real(Y).double().norm()) * 1e-2)
    del FhY
    torch.cuda.empty_cache()

    # linearity: F(2 x) = 2 F(x) bit for bit (a power of two scales exactly through every fp32 operation)
    x.mul_(2.0)
    F2 = plan.forward(x)
    assert torch.equal(torch.view_as_real(F2), 2.0 * torch.view_as_real(Fx))
    del F2, Fx
    torch.cuda.empty_cache()

    if w.C_in == w.C_out:
        g = x                                           # any real field serves as the upstream gradient
        y = plan.inverse(Y)
        GY = plan.backward_spectrum(g)
        lhs, rhs = rdot(y, g), cdot(Y, GY)
        scale = float(y.double().norm() * g.double().norm())
        assert abs(lhs - rhs) <= 2e-5 * max(abs(lhs), 1e-2 * scale)
    torch.cuda.synchronize()
    assert plan.status() == 0
    plan.close()
