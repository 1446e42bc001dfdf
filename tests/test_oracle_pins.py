"""Pins for the CPU oracle: each check is independent of the oracle's own formula.

numpy.fft (a different algorithm), closed forms, brute force on tiny grids, the
adjoint identity, Parseval, slab linearity, finite differences, torch float64
autograd through an FFT-based layer, and the paper's printed flop table.
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import dtst_oracle as O

RNG = np.random.default_rng(20260714)

TINY = [
    ((8,), (3,)),
    ((7,), (4,)),            # odd N, k = floor(N/2)+1
    ((8,), (5,)),            # includes Nyquist on the one-sided dim
    ((6, 8), (3, 2)),        # 2k = N on the two-sided dim
    ((5, 6), (1, 1)),        # k = 1
    ((8, 6, 10), (2, 3, 3)),
    ((4, 6, 5, 8), (2, 1, 2, 3)),
    ((6, 4, 4, 6), (3, 2, 1, 4)),   # 2k=N, Nyquist on last
]


def _rand_x(N, B=2, C=3):
    return RNG.standard_normal((B, C) + tuple(N))


def _rand_spec(N, kmax, B=2, C=2):
    K = [len(s) for s in O.mode_index_lists(N, kmax)]
    return RNG.standard_normal((B, C) + tuple(K)) + 1j * RNG.standard_normal((B, C) + tuple(K))


def _fft_slice(x, kmax):
    N = x.shape[2:]
    d = len(N)
    full = np.fft.rfftn(x, axes=tuple(range(2, 2 + d)))
    lists = O.mode_index_lists(N, kmax)
    return full[np.ix_(range(x.shape[0]), range(x.shape[1]), *lists)]


def _irfftn_padded(Y, N, kmax):
    d = len(N)
    lists = O.mode_index_lists(N, kmax)
    full = np.zeros(Y.shape[:2] + tuple(N[:-1]) + (N[-1] // 2 + 1,), dtype=np.complex128)
    full[np.ix_(range(Y.shape[0]), range(Y.shape[1]), *lists)] = Y
    return np.fft.irfftn(full, s=N, axes=tuple(range(2, 2 + d)))


# ---------------------------------------------------------------- mode set
def test_retained_indices_match_the_set_definition():
    # S_j = {0..k-1} U {N-k..N-1}: 8 low then 8 high for N=128, k=8 (the paper's figure).
    idx = O.retained_indices(128, 8, one_sided=False)
    assert idx.tolist() == list(range(8)) + list(range(120, 128))
    assert O.retained_indices(64, 8, one_sided=True).tolist() == list(range(8))
    with pytest.raises(ValueError):
        O.retained_indices(8, 5, one_sided=False)
    assert O.num_modes((128, 128, 128, 64), (16, 16, 16, 8)) == 262144


def test_retained_indices_equal_fft_slices():
    # cat(fft[:k], fft[-k:]) selects the same entries
    N, k = 12, 4
    v = np.arange(N)
    assert O.retained_indices(N, k, False).tolist() == np.concatenate([v[:k], v[-k:]]).tolist()


# ---------------------------------------------------------------- forward
@pytest.mark.parametrize("N,kmax", TINY)
def test_forward_separable_equals_literal_sum(N, kmax):
    x = _rand_x(N)
    a = O.forward(x, kmax)
    b = O.forward_literal(x, kmax)
    assert O.rel_l2(a, b) < 1e-12


@pytest.mark.parametrize("N,kmax", TINY)
def test_forward_equals_fft_then_truncate(N, kmax):
    x = _rand_x(N)
    assert O.rel_l2(O.forward(x, kmax), _fft_slice(x, kmax)) < 1e-12


def test_forward_literal_brute_force_python_loops():
    # a third, loop-only statement of Eq. 5 on a 3x4 grid
    N, kmax = (3, 4), (1, 2)
    x = _rand_x(N, 1, 1)
    lists = O.mode_index_lists(N, kmax)
    got = O.forward_literal(x, kmax)[0, 0]
    for a, s0 in enumerate(lists[0]):
        for b, s1 in enumerate(lists[1]):
            acc = 0j
            for n0 in range(N[0]):
                for n1 in range(N[1]):
                    acc += x[0, 0, n0, n1] * np.exp(-2j * np.pi * (s0 * n0 / N[0] + s1 * n1 / N[1]))
            assert abs(acc - got[a, b]) < 1e-12


def test_forward_closed_forms():
    N, kmax = (8, 6, 10), (2, 3, 3)
    lists = O.mode_index_lists(N, kmax)
    # delta at n0 -> unit-modulus phases e^{-i theta_m . n0}
    n0 = (3, 4, 7)
    x = np.zeros((1, 1) + N)
    x[(0, 0) + n0] = 1.0
    X = O.forward(x, kmax)[0, 0]
    for pos in itertools.product(*[range(len(s)) for s in lists]):
        th = sum(2 * np.pi * lists[j][pos[j]] * n0[j] / N[j] for j in range(3))
        assert abs(X[pos] - np.exp(-1j * th)) < 1e-13
    # constant field -> prod(N) at DC, zero elsewhere
    X = O.forward(np.ones((1, 1) + N), kmax)[0, 0]
    assert abs(X[0, 0, 0] - math.prod(N)) < 1e-10
    X[0, 0, 0] = 0
    assert np.abs(X).max() < 1e-10
    # a single retained cosine: x = cos(2 pi f.n/N + phi) -> (prod N / 2) e^{i phi} at f only
    f = (1, 5, 2)  # 5 = -1 on the N=6 axis; retained since k=3 keeps {0,1,2,3,4,5}
    phi = 0.7
    grids = np.meshgrid(*[np.arange(n) for n in N], indexing="ij")
    arg = sum(2 * np.pi * f[j] * grids[j] / N[j] for j in range(3)) + phi
    X = O.forward(np.cos(arg)[None, None], kmax)[0, 0]
    pos = tuple(int(np.where(lists[j] == f[j])[0][0]) for j in range(3))
    assert abs(X[pos] - math.prod(N) / 2 * np.exp(1j * phi)) < 1e-10
    X[pos] = 0
    assert np.abs(X).max() < 1e-10


def test_basis_matrix_offset_is_a_global_shift():
    # Eq. 18: the local basis of a rank is the global basis restricted to its columns
    N, k = 16, 3
    idx = O.retained_indices(N, k, False)
    full = O.basis_matrix(N, idx)
    part = O.basis_matrix(N, idx, n_local=4, offset=8)
    assert np.allclose(part, full[:, 8:12], atol=1e-15)
    # and each entry is the textbook twiddle
    assert abs(full[4, 5] - np.exp(-2j * np.pi * idx[4] * 5 / N)) < 1e-13


@pytest.mark.parametrize("N,kmax,P", [((8, 6, 10), (2, 3, 3), 4), ((8, 6, 10), (2, 3, 3), 8),
                                        ((12, 5), (3, 2), 3), ((4, 6, 5, 8), (2, 1, 2, 3), 2),
                                        ((16,), (5,), 4)])
def test_slab_partials_sum_to_the_whole(N, kmax, P):
    # Eq. 6-7, including N_0/P < K_0 and N_0/P = 1
    x = _rand_x(N)
    assert O.rel_l2(O.forward_sharded(x, kmax, P), _fft_slice(x, kmax)) < 1e-12


def test_pencil_offsets_on_two_dims():
    N, kmax = (8, 6, 10), (2, 3, 3)
    x = _rand_x(N, 1, 2)
    acc = 0
    for p0 in range(2):
        for p1 in range(3):
            blk = x[:, :, p0 * 4:(p0 + 1) * 4, p1 * 2:(p1 + 1) * 2]
            acc = acc + O.forward(blk, kmax, N_global=N, offsets=(p0 * 4, p1 * 2, 0))
    assert O.rel_l2(acc, _fft_slice(x, kmax)) < 1e-12


# ---------------------------------------------------------------- inverse
@pytest.mark.parametrize("N,kmax", TINY)
def test_inverse_equals_irfftn_of_zero_padded_spectrum(N, kmax):
    # random, NON-Hermitian spectrum: the f=0 / Nyquist imaginary parts are dropped like c2r
    Y = _rand_spec(N, kmax)
    ref = _irfftn_padded(Y, N, kmax)
    assert O.rel_l2(O.inverse(Y, N, kmax), ref) < 1e-12
    assert O.rel_l2(O.inverse_literal(Y, N, kmax), ref) < 1e-12


def test_inverse_local_block_is_a_slice_of_the_global_inverse():
    N, kmax = (8, 6, 10), (2, 3, 3)
    Y = _rand_spec(N, kmax)
    full = O.inverse(Y, N, kmax)
    part = O.inverse(Y, N, kmax, n_local=(2, 6, 10), offsets=(4, 0, 0))
    assert np.allclose(part, full[:, :, 4:6], atol=1e-14)


def test_hermitian_weights():
    assert O.hermitian_weights(8, 5).tolist() == [1, 2, 2, 2, 1]
    assert O.hermitian_weights(64, 8).tolist() == [1] + [2] * 7
    assert O.hermitian_weights(7, 4).tolist() == [1, 2, 2, 2]


def test_parseval_and_round_trip_on_band_limited_fields():
    N, kmax = (8, 6, 10), (3, 2, 4)
    Y = _rand_spec(N, kmax, 1, 2)
    # drop the unpaired -k frequency on the two-sided dims so the field is band-limited
    Y[:, :, kmax[0]] = 0
    Y[:, :, :, kmax[1]] = 0
    xb = O.inverse(Y, N, kmax)
    Xb = O.forward(xb, kmax)
    c = O.hermitian_weights(N[-1], kmax[-1])
    lhs = np.sum(xb ** 2)
    rhs = np.sum(c * np.abs(Xb) ** 2) / math.prod(N)
    assert abs(lhs - rhs) / lhs < 1e-12
    assert O.rel_l2(O.inverse(Xb, N, kmax), xb) < 1e-12


# ---------------------------------------------------------------- adjoints
@pytest.mark.parametrize("N,kmax", TINY)
def test_adjoint_identity(N, kmax):
    x = _rand_x(N, 1, 2)
    Y = _rand_spec(N, kmax, 1, 2)
    lhs = np.sum((np.conj(O.forward(x, kmax)) * Y).real)          # Re<F x, Y>
    rhs = np.sum(x * O.inverse(Y, N, kmax, doubling=False, normalise=False))   # <x, F^H Y>
    assert abs(lhs - rhs) <= 1e-12 * max(1.0, abs(lhs))


def test_adjoint_is_literal_sum():
    N, kmax = (4, 6), (2, 2)
    Y = _rand_spec(N, kmax, 1, 1)
    lists = O.mode_index_lists(N, kmax)
    got = O.inverse(Y, N, kmax, doubling=False, normalise=False)[0, 0]
    ref = np.zeros(N)
    for a, s0 in enumerate(lists[0]):
        for b, s1 in enumerate(lists[1]):
            for n0 in range(N[0]):
                for n1 in range(N[1]):
                    ref[n0, n1] += (Y[0, 0, a, b] * np.exp(2j * np.pi * (s0 * n0 / N[0] + s1 * n1 / N[1]))).real
    assert np.allclose(got, ref, atol=1e-12)


# ---------------------------------------------------------------- mixing
def test_mixing_identity_and_triple_loop():
    B, Ci, Co, M = 2, 3, 4, 5
    X = RNG.standard_normal((B, Ci, M)) + 1j * RNG.standard_normal((B, Ci, M))
    W = RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M))
    Y = O.spectral_mul(X, W)
    for b in range(B):
        for o in range(Co):
            for m in range(M):
                acc = sum(X[b, i, m] * W[i, o, m] for i in range(Ci))
                assert abs(acc - Y[b, o, m]) < 1e-13
    eye = np.zeros((Ci, Ci, M), dtype=complex)
    for i in range(Ci):
        eye[i, i] = 1
    assert np.allclose(O.spectral_mul(X, eye), X)


# ---------------------------------------------------------------- backward
def _torch_layer_grads(x, W, g, kmax):
    import torch
    N = x.shape[2:]
    d = len(N)
    dims = tuple(range(2, 2 + d))
    lists = O.mode_index_lists(N, kmax)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.complex128, requires_grad=True)
    Xf = torch.fft.rfftn(xt, dim=dims)
    ix = torch.meshgrid(*[torch.tensor(l) for l in lists], indexing="ij")
    Xs = Xf[(slice(None), slice(None)) + tuple(ix)]
    K = Xs.shape[2:]
    Ys = torch.einsum("bim,iom->bom", Xs.reshape(x.shape[0], x.shape[1], -1), Wt.reshape(W.shape[0], W.shape[1], -1))
    Ys = Ys.reshape((x.shape[0], W.shape[1]) + tuple(K))
    full = torch.zeros((x.shape[0], W.shape[1]) + tuple(N[:-1]) + (N[-1] // 2 + 1,), dtype=torch.complex128)
    full[(slice(None), slice(None)) + tuple(ix)] = Ys
    y = torch.fft.irfftn(full, s=N, dim=dims)
    (y * torch.tensor(g)).sum().backward()
    return y.detach().numpy(), xt.grad.numpy(), Wt.grad.numpy()


@pytest.mark.parametrize("N,kmax", [((8, 6, 10), (2, 3, 3)), ((4, 6, 5, 8), (2, 1, 2, 3)), ((6, 8), (3, 5))])
def test_layer_and_backward_match_torch_autograd(N, kmax):
    B, Ci, Co = 2, 3, 2
    x = _rand_x(N, B, Ci)
    M = O.num_modes(N, kmax)
    W = RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M))
    g = RNG.standard_normal((B, Co) + tuple(N))
    y_ref, gx_ref, gW_ref = _torch_layer_grads(x, W, g, kmax)
    y, Xhat = O.layer_forward(x, W, kmax)
    gx, gW = O.backward(g, Xhat, W, kmax)
    assert O.rel_l2(y, y_ref) < 1e-12
    assert O.rel_l2(gx, gx_ref) < 1e-12
    assert O.rel_l2(gW, gW_ref) < 1e-12


# ---------------------------------------------------------------- the complex primitive (two-sided on every dim)
@pytest.mark.parametrize("N,kmax", [((8,), (3,)), ((6, 8), (3, 2)), ((5, 6, 8), (2, 3, 4)), ((4, 6, 5, 8), (2, 1, 2, 3))])
def test_complex_forward_and_inverse_against_fftn(N, kmax):
    B, C = 2, 2
    x = RNG.standard_normal((B, C) + N) + 1j * RNG.standard_normal((B, C) + N)
    lists = O.mode_index_lists_complex(N, kmax)
    dims = tuple(range(2, 2 + len(N)))
    full = np.fft.fftn(x, axes=dims)
    want = full[(slice(None), slice(None)) + np.ix_(*lists)]
    X = O.forward_complex(x, kmax)
    assert X.shape == (B, C) + tuple(2 * k for k in kmax)
    assert O.rel_l2(X, want) < 1e-12
    # inverse: ifftn of the spectrum zero-padded outside the retained set
    Y = RNG.standard_normal(X.shape) + 1j * RNG.standard_normal(X.shape)
    pad = np.zeros((B, C) + N, dtype=complex)
    pad[(slice(None), slice(None)) + np.ix_(*lists)] = Y
    assert O.rel_l2(O.inverse_complex(Y, N, kmax), np.fft.ifftn(pad, axes=dims)) < 1e-12
    # slabs along dim 0 with global offsets sum to the whole (Eq. 6-7), and a block of the inverse is a slice
    if N[0] % 2 == 0:
        h = N[0] // 2
        parts = sum(O.forward_complex(x[:, :, p * h:(p + 1) * h], kmax, N_global=N, offsets=(p * h,) + (0,) * (len(N) - 1))
                    for p in range(2))
        assert O.rel_l2(parts, X) < 1e-12
        blk = O.inverse_complex(Y, N, kmax, n_local=(h,) + N[1:], offsets=(h,) + (0,) * (len(N) - 1))
        assert O.rel_l2(blk, O.inverse_complex(Y, N, kmax)[:, :, h:]) < 1e-12
    # a real field's complex transform agrees with the real path on the modes both keep (f >= 0 on the last dim)
    xr = RNG.standard_normal((B, C) + N)
    if kmax[-1] <= N[-1] // 2:
        assert O.rel_l2(O.forward_complex(xr, kmax)[..., :kmax[-1]], O.forward(xr, kmax)) < 1e-12


def test_complex_layer_backward_matches_torch_autograd():
    import torch
    N, kmax, B, Ci, Co = (6, 8, 10), (2, 3, 4), 2, 3, 2
    x = RNG.standard_normal((B, Ci) + N) + 1j * RNG.standard_normal((B, Ci) + N)
    M = int(np.prod([2 * k for k in kmax]))
    W = RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M))
    g = RNG.standard_normal((B, Co) + N) + 1j * RNG.standard_normal((B, Co) + N)
    y, Xhat = O.layer_forward_complex(x, W, kmax)
    gx, gW = O.backward_complex(g, Xhat, W, kmax)
    lists = O.mode_index_lists_complex(N, kmax)
    dims = tuple(range(2, 5))
    xt = torch.tensor(x, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    ix = torch.meshgrid(*[torch.tensor(l) for l in lists], indexing="ij")
    Xs = torch.fft.fftn(xt, dim=dims)[(slice(None), slice(None)) + tuple(ix)]
    Ys = torch.einsum("bim,iom->bom", Xs.reshape(B, Ci, -1), Wt)
    full = torch.zeros((B, Co) + N, dtype=torch.complex128)
    full[(slice(None), slice(None)) + tuple(ix)] = Ys.reshape((B, Co) + tuple(Xs.shape[2:]))
    yt = torch.fft.ifftn(full, dim=dims)
    gt = torch.tensor(g)
    (yt.real * gt.real + yt.imag * gt.imag).sum().backward()      # L with dL/dRe y = Re g, dL/dIm y = Im g
    assert O.rel_l2(y, yt.detach().numpy()) < 1e-12
    assert O.rel_l2(gx, xt.grad.numpy()) < 1e-12
    assert O.rel_l2(gW, Wt.grad.numpy()) < 1e-12


# ---------------------------------------------------------------- the whole block (bypass + GELU)
def test_gelu_against_math_erf_closed_forms_and_torch():
    import torch
    z = np.concatenate([np.linspace(-9, 9, 721), RNG.standard_normal(300) * 3])
    want = np.array([0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in z])
    assert np.max(np.abs(O.gelu(z) - want)) < 1e-15
    assert O.gelu(0.0) == 0.0
    assert np.allclose(O.gelu(z) - O.gelu(-z), z, atol=1e-14)          # z Phi(z) + z Phi(-z) = z
    assert abs(O.gelu(40.0) - 40.0) < 1e-12 and abs(O.gelu(-40.0)) < 1e-12
    t = torch.tensor(z, dtype=torch.float64, requires_grad=True)
    out = torch.nn.functional.gelu(t)                                  # exact (erf) form
    out.sum().backward()
    assert np.max(np.abs(O.gelu(z) - out.detach().numpy())) < 1e-14
    assert np.max(np.abs(O.gelu_grad(z) - t.grad.numpy())) < 1e-13
    h = 1e-6                                                           # and a central difference
    assert np.max(np.abs((O.gelu(z + h) - O.gelu(z - h)) / (2 * h) - O.gelu_grad(z))) < 1e-8


def test_bypass_is_a_pointwise_matrix_product():
    x = RNG.standard_normal((2, 3, 4, 5))
    Wb = RNG.standard_normal((2, 3))
    z = O.bypass(x, Wb)
    for b in range(2):
        for n0 in range(4):
            for n1 in range(5):
                assert np.allclose(z[b, :, n0, n1], Wb @ x[b, :, n0, n1])
    assert np.allclose(O.bypass(x[:, :, :, :], np.eye(3)), x)


def _torch_block_grads(x, W, Wb, g, kmax):
    import torch
    N = x.shape[2:]
    d = len(N)
    dims = tuple(range(2, 2 + d))
    lists = O.mode_index_lists(N, kmax)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.complex128, requires_grad=True)
    Wbt = torch.tensor(Wb, dtype=torch.float64, requires_grad=True)
    Xf = torch.fft.rfftn(xt, dim=dims)
    ix = torch.meshgrid(*[torch.tensor(l) for l in lists], indexing="ij")
    Xs = Xf[(slice(None), slice(None)) + tuple(ix)]
    K = Xs.shape[2:]
    Ys = torch.einsum("bim,iom->bom", Xs.reshape(x.shape[0], x.shape[1], -1), Wt.reshape(W.shape[0], W.shape[1], -1))
    full = torch.zeros((x.shape[0], W.shape[1]) + tuple(N[:-1]) + (N[-1] // 2 + 1,), dtype=torch.complex128)
    full[(slice(None), slice(None)) + tuple(ix)] = Ys.reshape((x.shape[0], W.shape[1]) + tuple(K))
    y = torch.fft.irfftn(full, s=N, dim=dims)
    lin = torch.nn.functional.linear(xt.movedim(1, -1), Wbt).movedim(-1, 1)     # a 1x1 convolution, no bias
    out = torch.nn.functional.gelu(lin + y)
    (out * torch.tensor(g)).sum().backward()
    return out.detach().numpy(), xt.grad.numpy(), Wt.grad.numpy(), Wbt.grad.numpy()


@pytest.mark.parametrize("N,kmax", [((8, 6, 10), (2, 3, 3)), ((4, 6, 5, 8), (2, 1, 2, 3)), ((6, 8), (3, 5))])
def test_block_forward_and_backward_match_torch_autograd(N, kmax):
    B, Ci, Co = 2, 3, 2
    x = _rand_x(N, B, Ci)
    M = O.num_modes(N, kmax)
    W = (RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M))) * 3.0
    Wb = RNG.standard_normal((Co, Ci))
    g = RNG.standard_normal((B, Co) + tuple(N))
    out_ref, gx_ref, gW_ref, gWb_ref = _torch_block_grads(x, W, Wb, g, kmax)
    out, z, Xhat = O.block_forward(x, W, Wb, kmax)
    gx, gW, gWb = O.block_backward(g, x, z, Xhat, W, Wb, kmax)
    assert O.rel_l2(out, out_ref) < 1e-12
    assert O.rel_l2(gx, gx_ref) < 1e-12
    assert O.rel_l2(gW, gW_ref) < 1e-12
    assert O.rel_l2(gWb, gWb_ref) < 1e-12
    # with the bypass and the activation switched off the block is the layer itself
    y, _ = O.layer_forward(x, W, kmax)
    _, z0, _ = O.block_forward(x, W, np.zeros_like(Wb), kmax)
    assert np.allclose(z0, y, atol=1e-13)


def test_block_backward_matches_finite_differences():
    N, kmax, B, Ci, Co = (4, 6), (2, 2), 1, 2, 2
    x = _rand_x(N, B, Ci)
    M = O.num_modes(N, kmax)
    W = (RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M)))
    Wb = RNG.standard_normal((Co, Ci))
    g = RNG.standard_normal((B, Co) + N)
    loss = lambda xx, ww, wb: float(np.sum(O.block_forward(xx, ww, wb, kmax)[0] * g))
    out, z, Xhat = O.block_forward(x, W, Wb, kmax)
    gx, gW, gWb = O.block_backward(g, x, z, Xhat, W, Wb, kmax)
    h = 1e-6
    for idx in [(0, 0, 1, 2), (0, 1, 3, 5)]:
        e = np.zeros_like(x)
        e[idx] = h
        assert abs((loss(x + e, W, Wb) - loss(x - e, W, Wb)) / (2 * h) - gx[idx]) < 1e-7
    for idx in [(0, 1), (1, 0)]:
        e = np.zeros_like(Wb)
        e[idx] = h
        assert abs((loss(x, W, Wb + e) - loss(x, W, Wb - e)) / (2 * h) - gWb[idx]) < 1e-7
    for idx in [(0, 1, 3), (1, 0, 5)]:
        e = np.zeros_like(W)
        e[idx] = h
        re = (loss(x, W + e, Wb) - loss(x, W - e, Wb)) / (2 * h)
        im = (loss(x, W + 1j * e, Wb) - loss(x, W - 1j * e, Wb)) / (2 * h)
        assert abs(re - gW[idx].real) < 1e-7 and abs(im - gW[idx].imag) < 1e-7


def test_fno_forward_and_backward_match_torch_autograd():
    """A whole small FNO (lift, two Fourier layers, projection) against torch float64 autograd through
    rfftn / irfftn, linear layers and the exact GELU."""
    import torch
    N, kmax, B, Ca, dv, Cu, L = (6, 8, 10), (2, 3, 4), 2, 3, 4, 2, 2
    M = O.num_modes(N, kmax)
    a = _rand_x(N, B, Ca)
    params = {"P_w": RNG.standard_normal((dv, Ca)), "P_b": RNG.standard_normal(dv),
              "blocks": [((RNG.standard_normal((dv, dv, M)) + 1j * RNG.standard_normal((dv, dv, M))),
                          RNG.standard_normal((dv, dv)) / 2) for _ in range(L)],
              "Q_w": RNG.standard_normal((Cu, dv)), "Q_b": RNG.standard_normal(Cu)}
    g = RNG.standard_normal((B, Cu) + N)
    u, saved = O.fno_forward(a, params, kmax)
    grads = O.fno_backward(g, params, saved, kmax)

    d = len(N)
    dims = tuple(range(2, 2 + d))
    lists = O.mode_index_lists(N, kmax)
    ix = torch.meshgrid(*[torch.tensor(l) for l in lists], indexing="ij")
    t = lambda v, c=False: torch.tensor(v, dtype=torch.complex128 if c else torch.float64, requires_grad=True)
    at, Pw, Pb, Qw, Qb = t(a), t(params["P_w"]), t(params["P_b"]), t(params["Q_w"]), t(params["Q_b"])
    Ws = [(t(W, True), t(Wb)) for W, Wb in params["blocks"]]
    lin = lambda x, w, b=None: torch.nn.functional.linear(x.movedim(1, -1), w, b).movedim(-1, 1)
    v = lin(at, Pw, Pb)
    for W, Wb in Ws:
        Xs = torch.fft.rfftn(v, dim=dims)[(slice(None), slice(None)) + tuple(ix)]
        Ys = torch.einsum("bim,iom->bom", Xs.reshape(B, dv, -1), W)
        full = torch.zeros((B, dv) + tuple(N[:-1]) + (N[-1] // 2 + 1,), dtype=torch.complex128)
        full[(slice(None), slice(None)) + tuple(ix)] = Ys.reshape((B, dv) + tuple(Xs.shape[2:]))
        v = torch.nn.functional.gelu(lin(v, Wb) + torch.fft.irfftn(full, s=N, dim=dims))
    ut = lin(v, Qw, Qb)
    (ut * torch.tensor(g)).sum().backward()
    assert O.rel_l2(u, ut.detach().numpy()) < 1e-12
    assert O.rel_l2(grads["a"], at.grad.numpy()) < 1e-11
    for name, tt in (("P_w", Pw), ("P_b", Pb), ("Q_w", Qw), ("Q_b", Qb)):
        assert O.rel_l2(grads[name], tt.grad.numpy()) < 1e-11, name
    for l in range(L):
        assert O.rel_l2(grads["blocks"][l][0], Ws[l][0].grad.numpy()) < 1e-11
        assert O.rel_l2(grads["blocks"][l][1], Ws[l][1].grad.numpy()) < 1e-11


def test_block_layer_and_backward_are_slices_and_sums_of_the_global_ones():
    # a rank's block (Eq. 18): y and grad_x of the block are slices of the global results when the
    # block's spectrum is replaced by the summed one; partial spectra and grad_W sum over blocks
    N, kmax = (8, 6, 10), (2, 3, 3)
    B, Ci, Co = 1, 2, 2
    x = _rand_x(N, B, Ci)
    M = O.num_modes(N, kmax)
    W = RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M))
    g = RNG.standard_normal((B, Co) + tuple(N))
    y, Xhat = O.layer_forward(x, W, kmax)
    gx, gW = O.backward(g, Xhat, W, kmax)
    Xsum, gWsum, GY_parts = 0, 0, []
    for p in range(4):
        sl = slice(2 * p, 2 * p + 2)
        off = (2 * p, 0, 0)
        yb, Xp = O.layer_forward(x[:, :, sl], W, kmax, N_global=N, offsets=off)
        Xsum = Xsum + Xp
        _, gWp = O.backward(g[:, :, sl], Xhat, W, kmax, N_global=N, offsets=off)
        gWsum = gWsum + gWp
    assert O.rel_l2(Xsum, Xhat) < 1e-12
    assert O.rel_l2(gWsum, gW) < 1e-12
    # block inverse of the global spectrum is the slice of the global inverse
    Y = O.spectral_mul(Xhat, W.reshape((Ci, Co) + Xhat.shape[2:]))
    yb = O.inverse(Y, N, kmax, n_local=(2, 6, 10), offsets=(4, 0, 0))
    assert np.allclose(yb, y[:, :, 4:6], atol=1e-13)


def test_backward_matches_finite_differences():
    N, kmax = (4, 6), (2, 2)
    B, Ci, Co = 1, 2, 2
    x = _rand_x(N, B, Ci)
    M = O.num_modes(N, kmax)
    W = RNG.standard_normal((Ci, Co, M)) + 1j * RNG.standard_normal((Ci, Co, M))
    g = RNG.standard_normal((B, Co) + tuple(N))

    def loss(xx, WW):
        return float(np.sum(O.layer_forward(xx, WW, kmax)[0] * g))

    _, Xhat = O.layer_forward(x, W, kmax)
    gx, gW = O.backward(g, Xhat, W, kmax)
    h = 1e-6
    for idx in [(0, 0, 1, 2), (0, 1, 3, 5), (0, 1, 0, 0)]:
        xp, xm = x.copy(), x.copy()
        xp[idx] += h
        xm[idx] -= h
        fd = (loss(xp, W) - loss(xm, W)) / (2 * h)
        assert abs(fd - gx[idx]) < 1e-7 * max(1.0, abs(fd))
    for idx in [(0, 0, 0), (1, 1, 7), (0, 1, 3)]:
        for part, unit in ((np.real, 1.0), (np.imag, 1j)):
            Wp, Wm = W.copy(), W.copy()
            Wp[idx] += h * unit
            Wm[idx] -= h * unit
            fd = (loss(x, Wp) - loss(x, Wm)) / (2 * h)
            assert abs(fd - part(gW[idx])) < 1e-7 * max(1.0, abs(fd))


# ---------------------------------------------------------------- the paper's printed table
def test_flop_model_reproduces_table2():
    path = os.path.join(os.path.dirname(__file__), "golden", "table2_gemm_flops.txt")
    gold = {}
    with open(path) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                key, val = line.split()
                gold[key] = float(val)
    shape = (128, 128, 64, 30)          # X, Y, Z, T
    K = (16, 16, 16, 16)
    stages = O.gemm_flops_per_stage(shape, order=(3, 2, 1, 0), K=K, channels=20)
    got = [s / 1e9 for s in stages]
    for val, key in zip(got, ("stage_T", "stage_Z", "stage_Y", "stage_X")):
        assert abs(val - gold[key]) <= 0.05 + 1e-9, (key, val)
    assert abs(sum(got) - gold["total_gemm"]) <= 0.1
    fft = O.fft_flops(shape, 20) / 1e9
    assert abs(fft - gold["total_cufft"]) <= 0.1
    assert abs(sum(got) / fft - gold["ratio"]) <= 0.01
