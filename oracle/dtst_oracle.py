"""CPU oracle for the truncated spectral layer (TEST INFRASTRUCTURE ONLY).

A plain, slow, float64 numpy statement of what the layer computes, written from
the paper's definitions.  It shares no code with the CUDA path and must never be
imported by it: only the tests, the smoke check and the benchmark's CPU-baseline
leg may call into this package.

Conventions (d transformed dims, grid N = (N_0..N_{d-1}), last one contiguous):
  * dims 0..d-2 are two-sided: retained index list [0..k-1, N-k..N-1]
    (Section "Background and Motivation", definition of S_j);
  * dim d-1 is one-sided (the rfft dimension of a real field): [0..k-1];
  * forward sign e^{-2 pi i k n / N}, un-normalised (Eq. 5);
  * inverse sign +, scaled by 1/prod(N) (Eq. 14), real output with Hermitian
    doubling on the one-sided dimension (c2r semantics).

Every function below is pinned by tests that do not re-use its own formula:
numpy.fft (rfftn-then-slice, irfftn of the zero-padded spectrum), closed forms,
brute force on tiny grids, the adjoint identity, Parseval, slab linearity,
finite differences and torch float64 autograd (the block of Algorithm 1 with
its bypass and GELU included).  Nothing here is "parity unpinned".
"""
from __future__ import annotations

import itertools
import math

import numpy as np


# --------------------------------------------------------------------------
# Retained mode set (Section "Background and Motivation": S_j; Fig. "basis-matrix")
# --------------------------------------------------------------------------
def retained_indices(N: int, k: int, one_sided: bool) -> np.ndarray:
    """DFT indices kept along one dimension, ascending.

    Two-sided: [0..k-1] followed by [N-k..N-1] (2k entries); one-sided: [0..k-1].
    """
    if one_sided:
        if not (1 <= k <= N // 2 + 1):
            raise ValueError("one-sided k out of range")
        return np.arange(k, dtype=np.int64)
    if not (1 <= k and 2 * k <= N):
        raise ValueError("two-sided k out of range (needs 2k <= N)")
    return np.concatenate([np.arange(k, dtype=np.int64), np.arange(N - k, N, dtype=np.int64)])


def mode_index_lists(N, kmax):
    d = len(N)
    return [retained_indices(int(N[j]), int(kmax[j]), one_sided=(j == d - 1)) for j in range(d)]


def num_modes(N, kmax) -> int:
    return math.prod(len(s) for s in mode_index_lists(N, kmax))


# --------------------------------------------------------------------------
# Basis matrix with global phase offset (Eq. 18)
# --------------------------------------------------------------------------
def basis_matrix(N_global: int, idx: np.ndarray, n_local: int | None = None, offset: int = 0) -> np.ndarray:
    """B[s, j] = W_N^{idx[s] * (offset + j)}, W_N = e^{-2 pi i / N}; shape [len(idx), n_local].

    The integer product is reduced mod N before any floating-point operation.
    """
    n_local = N_global if n_local is None else n_local
    j = np.arange(n_local, dtype=np.int64) + int(offset)
    r = np.mod(np.outer(np.asarray(idx, dtype=np.int64), j), N_global)
    return np.exp(-2j * np.pi * r.astype(np.float64) / float(N_global))


# --------------------------------------------------------------------------
# Forward partial DFT, tier (i): the literal un-factored sum of Eq. 5/6
# --------------------------------------------------------------------------
def phase_tensor(N_global, modes, n_local=None, offsets=None) -> np.ndarray:
    """prod_j W_{N_j}^{s_j (off_j + n_j)} over the local grid, for one mode tuple."""
    d = len(N_global)
    n_local = tuple(N_global) if n_local is None else tuple(n_local)
    offsets = (0,) * d if offsets is None else tuple(offsets)
    ph = np.ones((), dtype=np.complex128)
    for j in range(d):
        n = np.arange(n_local[j], dtype=np.int64) + offsets[j]
        r = np.mod(int(modes[j]) * n, N_global[j]).astype(np.float64)
        f = np.exp(-2j * np.pi * r / N_global[j])
        shape = [1] * d
        shape[j] = n_local[j]
        ph = ph * f.reshape(shape)
    return ph


def forward_one_mode(x_c: np.ndarray, N_global, modes, offsets=None) -> complex:
    """Xhat at one retained mode for one real channel x_c[n_local...] (Eq. 5 as written)."""
    ph = phase_tensor(N_global, modes, x_c.shape, offsets)
    return complex(np.sum(x_c.astype(np.float64) * ph))


def forward_literal(x: np.ndarray, kmax, N_global=None, offsets=None) -> np.ndarray:
    """Xhat[B, C, K_0..K_{d-1}] by the un-factored sum; O(prod(N) * M): tiny grids only."""
    B, C = x.shape[:2]
    n_local = x.shape[2:]
    N_global = tuple(n_local) if N_global is None else tuple(N_global)
    lists = mode_index_lists(N_global, kmax)
    out = np.zeros((B, C) + tuple(len(s) for s in lists), dtype=np.complex128)
    x64 = x.astype(np.float64)
    for pos in itertools.product(*[range(len(s)) for s in lists]):
        modes = [lists[j][pos[j]] for j in range(len(lists))]
        ph = phase_tensor(N_global, modes, n_local, offsets)
        out[(slice(None), slice(None)) + pos] = np.sum(x64 * ph, axis=tuple(range(2, x.ndim)))
    return out


# --------------------------------------------------------------------------
# Forward partial DFT, tier (ii): separable, one dimension at a time
# (Section "Computing the Local Partial Spectrum")
# --------------------------------------------------------------------------
def _apply_along(mat: np.ndarray, t: np.ndarray, axis: int) -> np.ndarray:
    """out[..., r, ...] = sum_q mat[r, q] * t[..., q, ...] along `axis`."""
    return np.moveaxis(np.tensordot(mat, t, axes=([1], [axis])), 0, axis)


def forward(x: np.ndarray, kmax, N_global=None, offsets=None) -> np.ndarray:
    """Xhat[B, C, K_0..K_{d-1}] complex128 from real x[B, C, n_local...].

    Last dimension first, dimension 0 last (the order of Algorithm 1, line 2).
    With N_global/offsets given, x is one rank's block and the result is that
    rank's partial spectrum (Eq. 6).
    """
    n_local = x.shape[2:]
    d = len(n_local)
    N_global = tuple(n_local) if N_global is None else tuple(N_global)
    offsets = (0,) * d if offsets is None else tuple(offsets)
    lists = mode_index_lists(N_global, kmax)
    t = x.astype(np.complex128)
    for j in range(d - 1, -1, -1):
        Bj = basis_matrix(N_global[j], lists[j], n_local[j], offsets[j])
        t = _apply_along(Bj, t, 2 + j)
    return t


def forward_sharded(x: np.ndarray, kmax, P: int) -> np.ndarray:
    """Sum over P slabs along dim 0 of the slab partial spectra, ascending p (Eq. 6-7)."""
    N = x.shape[2:]
    if N[0] % P:
        raise ValueError("P must divide N_0")
    nl = N[0] // P
    acc = None
    for p in range(P):
        slab = x[:, :, p * nl:(p + 1) * nl]
        off = (p * nl,) + (0,) * (len(N) - 1)
        part = forward(slab, kmax, N_global=N, offsets=off)
        acc = part if acc is None else acc + part
    return acc


# --------------------------------------------------------------------------
# Per-mode channel mixing (Eq. 12, with index order out[b,o,m] = sum_i X[b,i,m] W[i,o,m])
# --------------------------------------------------------------------------
def spectral_mul(Xhat: np.ndarray, W: np.ndarray) -> np.ndarray:
    B, Ci = Xhat.shape[:2]
    Xf = Xhat.reshape(B, Ci, -1).astype(np.complex128)
    Wf = W.reshape(W.shape[0], W.shape[1], -1).astype(np.complex128)
    Y = np.einsum("bim,iom->bom", Xf, Wf)
    return Y.reshape((B, W.shape[1]) + Xhat.shape[2:])


# --------------------------------------------------------------------------
# Inverse partial DFT with Hermitian doubling (Eq. 14; B^{-1} = B^H / N)
# --------------------------------------------------------------------------
def hermitian_weights(N_last: int, k_last: int) -> np.ndarray:
    """c(f) on the one-sided dimension: 1 at f = 0 and at Nyquist (2f = N), else 2."""
    c = np.full(k_last, 2.0)
    c[0] = 1.0
    for f in range(k_last):
        if 2 * f == N_last:
            c[f] = 1.0
    return c


def inverse(Yhat: np.ndarray, N_global, kmax, n_local=None, offsets=None,
            doubling: bool = True, normalise: bool = True) -> np.ndarray:
    """y[B, C, n_local...] float64 = (1/prod N) sum_m c(m) Re(Yhat[m] prod_j W_{N_j}^{-s_j n_j}).

    Dimension 0 first, last dimension last (Algorithm 1, line 7).  With
    doubling=False and normalise=False this is the plain adjoint of `forward`.
    """
    d = len(N_global)
    N_global = tuple(N_global)
    n_local = N_global if n_local is None else tuple(n_local)
    offsets = (0,) * d if offsets is None else tuple(offsets)
    lists = mode_index_lists(N_global, kmax)
    t = Yhat.astype(np.complex128)
    if doubling:
        c = hermitian_weights(N_global[-1], int(kmax[-1]))
        t = t * c  # broadcasts over the last (one-sided) axis
    for j in range(d):
        Bj = basis_matrix(N_global[j], lists[j], n_local[j], offsets[j])
        t = _apply_along(Bj.conj().T, t, 2 + j)
    y = t.real
    if normalise:
        y = y / float(math.prod(N_global))
    return y


def inverse_literal(Yhat: np.ndarray, N_global, kmax) -> np.ndarray:
    """The same inverse as one un-factored sum over modes; tiny grids only."""
    N_global = tuple(N_global)
    lists = mode_index_lists(N_global, kmax)
    c = hermitian_weights(N_global[-1], int(kmax[-1]))
    B, C = Yhat.shape[:2]
    y = np.zeros((B, C) + N_global, dtype=np.float64)
    for pos in itertools.product(*[range(len(s)) for s in lists]):
        modes = [lists[j][pos[j]] for j in range(len(lists))]
        ph = np.conj(phase_tensor(N_global, modes))
        coef = Yhat[(slice(None), slice(None)) + pos].astype(np.complex128)
        y += c[pos[-1]] * np.real(coef.reshape(B, C, *([1] * len(N_global))) * ph)
    return y / float(math.prod(N_global))


# --------------------------------------------------------------------------
# The DTST primitive as the paper states it (Section "Distributed Truncated Spectral Transforms"): a COMPLEX
# d-dimensional tensor and the two-sided retained set S_j on EVERY dimension, the last one included
# (K_j = 2 k_j for all j).  No Hermitian symmetry, hence no doubling: the inverse is the plain complex sum of Eq. 14.
# --------------------------------------------------------------------------
def mode_index_lists_complex(N, kmax):
    return [retained_indices(int(N[j]), int(kmax[j]), one_sided=False) for j in range(len(N))]


def forward_complex(x: np.ndarray, kmax, N_global=None, offsets=None) -> np.ndarray:
    """Xhat[B, C, 2k_0..2k_{d-1}] from complex x[B, C, n_local...] (Eq. 5-6 with the basis of Eq. 18)."""
    n_local = x.shape[2:]
    d = len(n_local)
    N_global = tuple(n_local) if N_global is None else tuple(N_global)
    offsets = (0,) * d if offsets is None else tuple(offsets)
    lists = mode_index_lists_complex(N_global, kmax)
    t = x.astype(np.complex128)
    for j in range(d - 1, -1, -1):
        t = _apply_along(basis_matrix(N_global[j], lists[j], n_local[j], offsets[j]), t, 2 + j)
    return t


def inverse_complex(Yhat: np.ndarray, N_global, kmax, n_local=None, offsets=None, normalise: bool = True) -> np.ndarray:
    """y[B, C, n_local...] complex = (1/prod N) sum_m Yhat[m] prod_j W_{N_j}^{-s_j n_j} (Eq. 14, B^{-1} = B^H / N)."""
    d = len(N_global)
    N_global = tuple(N_global)
    n_local = N_global if n_local is None else tuple(n_local)
    offsets = (0,) * d if offsets is None else tuple(offsets)
    lists = mode_index_lists_complex(N_global, kmax)
    t = Yhat.astype(np.complex128)
    for j in range(d):
        t = _apply_along(basis_matrix(N_global[j], lists[j], n_local[j], offsets[j]).conj().T, t, 2 + j)
    return t / float(math.prod(N_global)) if normalise else t


def layer_forward_complex(x: np.ndarray, W: np.ndarray, kmax, N_global=None, offsets=None):
    n_local = x.shape[2:]
    N = tuple(n_local) if N_global is None else tuple(N_global)
    Xhat = forward_complex(x, kmax, N_global=N, offsets=offsets)
    Yhat = spectral_mul(Xhat, W.reshape((W.shape[0], W.shape[1]) + Xhat.shape[2:]))
    return inverse_complex(Yhat, N, kmax, n_local=n_local, offsets=offsets), Xhat


def backward_complex(grad_y: np.ndarray, Xhat: np.ndarray, W: np.ndarray, kmax, N_global=None, offsets=None):
    """Gradients of a real loss with upstream gradient grad_y = dL/dRe(y) + i dL/dIm(y) (the same convention for
    every complex quantity): each linear step is replaced by its adjoint (Section "Backward Pass")."""
    n_local = grad_y.shape[2:]
    N = tuple(n_local) if N_global is None else tuple(N_global)
    B = grad_y.shape[0]
    G_Y = forward_complex(grad_y, kmax, N_global=N, offsets=offsets) / float(math.prod(N))
    Ci, Co = W.shape[:2]
    Wm = W.reshape(Ci, Co, -1).astype(np.complex128)
    GYf = G_Y.reshape(B, Co, -1)
    Xf = Xhat.reshape(B, Ci, -1).astype(np.complex128)
    G_X = np.einsum("bom,iom->bim", GYf, Wm.conj())
    G_W = np.einsum("bim,bom->iom", Xf.conj(), GYf)
    g_x = inverse_complex(G_X.reshape((B, Ci) + G_Y.shape[2:]), N, kmax, n_local=n_local, offsets=offsets,
                          normalise=False)
    return g_x, G_W.reshape(W.shape)


# --------------------------------------------------------------------------
# The whole layer and its backward pass (Section "Backward Pass": adjoints)
# --------------------------------------------------------------------------
def layer_forward(x: np.ndarray, W: np.ndarray, kmax, N_global=None, offsets=None):
    """Returns (y, Xhat): y = I(M(F(x), W)); Xhat is what backward needs.

    With N_global/offsets, x is one rank's block: Xhat is its partial spectrum and
    y the block of the inverse of M(Xhat) (every step is linear, Eq. 6-7).
    """
    n_local = x.shape[2:]
    N = tuple(n_local) if N_global is None else tuple(N_global)
    Xhat = forward(x, kmax, N_global=N, offsets=offsets)
    Wm = W.reshape((W.shape[0], W.shape[1]) + Xhat.shape[2:])
    Yhat = spectral_mul(Xhat, Wm)
    return inverse(Yhat, N, kmax, n_local=n_local, offsets=offsets), Xhat


def backward(grad_y: np.ndarray, Xhat: np.ndarray, W: np.ndarray, kmax, N_global=None, offsets=None):
    """Gradients of L = sum(y * grad_y) w.r.t. x and W (complex gradient = dL/dRe + i dL/dIm).

    G_Yhat = (c / prod N) F(grad_y)                    adjoint of the inverse
    G_Xhat[b,i,m] = sum_o G_Yhat[b,o,m] conj(W[i,o,m])  adjoint of the mixing
    G_W[i,o,m]    = sum_b conj(Xhat[b,i,m]) G_Yhat[b,o,m]
    g_x = Re sum_m G_Xhat[m] e^{+i theta_m n}           adjoint of the forward
    """
    n_local = grad_y.shape[2:]
    N = tuple(n_local) if N_global is None else tuple(N_global)
    B = grad_y.shape[0]
    c = hermitian_weights(N[-1], int(kmax[-1]))
    G_Y = forward(grad_y, kmax, N_global=N, offsets=offsets) * c / float(math.prod(N))
    Ci, Co = W.shape[:2]
    Wm = W.reshape(Ci, Co, -1).astype(np.complex128)
    GYf = G_Y.reshape(B, Co, -1)
    Xf = Xhat.reshape(B, Ci, -1).astype(np.complex128)
    G_X = np.einsum("bom,iom->bim", GYf, Wm.conj())
    G_W = np.einsum("bim,bom->iom", Xf.conj(), GYf)
    g_x = inverse(G_X.reshape((B, Ci) + G_Y.shape[2:]), N, kmax, n_local=n_local, offsets=offsets,
                  doubling=False, normalise=False)
    return g_x, G_W.reshape(W.shape)


# --------------------------------------------------------------------------
# The whole block (Section "Block Structure", Algorithm 1 lines 1 and 8; Eq. 1):
#     x_next = GELU(W_bypass x + y),   y = I(M(F(x), W))
# W_bypass is the point-wise linear operator: [C_out, C_in], applied at every grid point; no bias is mentioned in
# the paper and none is applied.  GELU is the exact (erf) form, z Phi(z).
# --------------------------------------------------------------------------
def _erf(z: np.ndarray) -> np.ndarray:
    from scipy.special import erf      # a library primitive as one step; pinned against math.erf and torch
    return erf(z)


def gelu(z: np.ndarray) -> np.ndarray:
    """GELU(z) = z * Phi(z) = z/2 * (1 + erf(z / sqrt 2))."""
    z = np.asarray(z, dtype=np.float64)
    return 0.5 * z * (1.0 + _erf(z / math.sqrt(2.0)))


def gelu_grad(z: np.ndarray) -> np.ndarray:
    """d GELU / dz = Phi(z) + z * phi(z), phi the standard normal density."""
    z = np.asarray(z, dtype=np.float64)
    return 0.5 * (1.0 + _erf(z / math.sqrt(2.0))) + z * np.exp(-0.5 * z * z) / math.sqrt(2.0 * math.pi)


def bypass(x: np.ndarray, Wb: np.ndarray) -> np.ndarray:
    """(W_bypass x)[b, o, n] = sum_i Wb[o, i] x[b, i, n]  (Algorithm 1 line 1)."""
    return np.einsum("oi,bi...->bo...", np.asarray(Wb, dtype=np.float64), np.asarray(x, dtype=np.float64))


def block_forward(x: np.ndarray, W: np.ndarray, Wb: np.ndarray, kmax, N_global=None, offsets=None):
    """Returns (out, z, Xhat): z = W_bypass x + I(M(F(x), W)) is the pre-activation, out = GELU(z)
    (Algorithm 1 lines 1-8 without the collectives; with N_global/offsets, x is one rank's block and Xhat its
    partial spectrum, so z and out are only meaningful once the partial spectra have been summed)."""
    y, Xhat = layer_forward(x, W, kmax, N_global=N_global, offsets=offsets)
    z = bypass(x, Wb) + y
    return gelu(z), z, Xhat


def block_backward(grad_out: np.ndarray, x: np.ndarray, z: np.ndarray, Xhat: np.ndarray, W: np.ndarray,
                   Wb: np.ndarray, kmax, N_global=None, offsets=None):
    """Gradients of L = sum(out * grad_out) w.r.t. x, W (spectral) and W_bypass.

    g_z = grad_out * GELU'(z)                                  adjoint of the activation
    grad_Wb[o, i] = sum_{b, n} g_z[b, o, n] x[b, i, n]         the bypass is linear in Wb
    grad_x = Wb^T g_z + (adjoint of the spectral layer)(g_z)   (Section "Backward Pass")
    """
    gz = np.asarray(grad_out, dtype=np.float64) * gelu_grad(z)
    gx_spec, gW = backward(gz, Xhat, W, kmax, N_global=N_global, offsets=offsets)
    xb = np.asarray(x, dtype=np.float64)
    B = xb.shape[0]
    gWb = np.einsum("bon,bin->oi", gz.reshape(B, gz.shape[1], -1), xb.reshape(B, xb.shape[1], -1))
    gx = np.einsum("oi,bo...->bi...", np.asarray(Wb, dtype=np.float64), gz) + gx_spec
    return gx, gW, gWb


# --------------------------------------------------------------------------
# A whole Fourier neural operator (Section "Background and Motivation": the input is lifted to d_v channels by a
# point-wise network P, passed through L Fourier layers (Eq. 1) and projected back by a point-wise network Q).
# P and Q are taken as one linear map with bias each; every Fourier layer is the block above, activation included.
# params = {"P_w": [d_v, C_a], "P_b": [d_v], "blocks": [(W_l [d_v, d_v, M] complex, Wb_l [d_v, d_v]), ...],
#           "Q_w": [C_u, d_v], "Q_b": [C_u]}
# --------------------------------------------------------------------------
def pointwise_linear(x: np.ndarray, W: np.ndarray, b=None) -> np.ndarray:
    y = bypass(x, W)
    if b is not None:
        y = y + np.asarray(b, dtype=np.float64).reshape((1, -1) + (1,) * (x.ndim - 2))
    return y


def fno_forward(a: np.ndarray, params: dict, kmax):
    """Returns (u, saved): u = Q(block_L(... block_1(P(a)))), saved = what fno_backward needs."""
    v = pointwise_linear(a, params["P_w"], params["P_b"])
    saved = {"a": np.asarray(a, dtype=np.float64), "v": [], "z": [], "Xhat": []}
    for (W, Wb) in params["blocks"]:
        out, z, Xhat = block_forward(v, W, Wb, kmax)
        saved["v"].append(v)
        saved["z"].append(z)
        saved["Xhat"].append(Xhat)
        v = out
    saved["v_last"] = v
    return pointwise_linear(v, params["Q_w"], params["Q_b"]), saved


def fno_backward(grad_u: np.ndarray, params: dict, saved: dict, kmax) -> dict:
    """Gradients of L = sum(u * grad_u) w.r.t. every parameter (and the input a)."""
    g = np.asarray(grad_u, dtype=np.float64)
    B = g.shape[0]
    flat = lambda t: t.reshape(B, t.shape[1], -1)
    grads = {"Q_w": np.einsum("bon,bin->oi", flat(g), flat(saved["v_last"])), "Q_b": flat(g).sum(axis=(0, 2)),
             "blocks": [None] * len(params["blocks"])}
    g = bypass(g, np.asarray(params["Q_w"]).T)
    for l in reversed(range(len(params["blocks"]))):
        W, Wb = params["blocks"][l]
        g, gW, gWb = block_backward(g, saved["v"][l], saved["z"][l], saved["Xhat"][l], W, Wb, kmax)
        grads["blocks"][l] = (gW, gWb)
    grads["P_w"] = np.einsum("bon,bin->oi", flat(g), flat(saved["a"]))
    grads["P_b"] = flat(g).sum(axis=(0, 2))
    grads["a"] = bypass(g, np.asarray(params["P_w"]).T)
    return grads


# --------------------------------------------------------------------------
# Flop model of the per-dimension gemm pipeline (Table 2)
# --------------------------------------------------------------------------
def gemm_flops_per_stage(shape, order, K, channels: int):
    """2*K*N flops per 1-D transform of length N, applied to every line of the
    progressively compressed tensor, in the given contraction order."""
    cur = list(shape)
    out = []
    for ax in order:
        lines = channels * math.prod(cur) // cur[ax]
        out.append(2.0 * K[ax] * cur[ax] * lines)
        cur[ax] = K[ax]
    return out


def fft_flops(shape, channels: int) -> float:
    """(5/2) N log2 N per 1-D FFT, all dimensions, no compression."""
    total = channels * math.prod(shape)
    return sum(2.5 * total * math.log2(n) for n in shape)


def rel_l2(a: np.ndarray, ref: np.ndarray) -> float:
    """||a - ref||_2 / ||ref||_2 over the whole tensor, complex as two reals, in float64."""
    a = np.asarray(a)
    ref = np.asarray(ref)
    num = np.linalg.norm((a.astype(np.complex128) - ref.astype(np.complex128)).ravel())
    den = np.linalg.norm(ref.astype(np.complex128).ravel())
    return float(num / den) if den > 0 else float(num)
