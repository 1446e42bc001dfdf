"""Property-based pins of the oracle (hypothesis): on shapes nobody chose by hand the float64 statement must keep the
identities that the mathematics fixes - agreement with the library FFT, linearity over slabs (Eq. 6-7), the adjoint
identity, and the step-wise backward (spectrum -> mixing adjoint -> input) being the gradient of L = sum(y * g) as
torch's autograd computes it through rfftn / irfftn."""
import math

import numpy as np
import pytest
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from oracle import dtst_oracle as O


@st.composite
def layer_shapes(draw):
    d = draw(st.integers(1, 3))
    N = [draw(st.integers(2, 9)) for _ in range(d - 1)] + [draw(st.integers(2, 10))]
    k = [draw(st.integers(1, max(1, n // 2))) for n in N[:-1]] + [draw(st.integers(1, N[-1] // 2 + 1))]
    return tuple(N), tuple(k)


SETTINGS = dict(max_examples=40, deadline=None, suppress_health_check=[HealthCheck.too_slow])


@settings(**SETTINGS)
@given(layer_shapes(), st.integers(0, 2 ** 31 - 1))
def test_forward_is_the_truncated_library_fft(shape, seed):
    N, k = shape
    x = np.random.default_rng(seed).standard_normal((1, 2) + N)
    full = np.fft.rfftn(x, axes=tuple(range(2, 2 + len(N))))
    idx = np.ix_(*O.mode_index_lists(N, k))
    ref = full[(slice(None), slice(None)) + idx]
    assert O.rel_l2(O.forward(x, k), ref) < 1e-12


@settings(**SETTINGS)
@given(layer_shapes(), st.integers(0, 2 ** 31 - 1))
def test_inverse_is_irfftn_of_the_zero_padded_spectrum(shape, seed):
    N, k = shape
    rng = np.random.default_rng(seed)
    K = tuple(len(l) for l in O.mode_index_lists(N, k))
    Y = rng.standard_normal((1, 2) + K) + 1j * rng.standard_normal((1, 2) + K)
    full = np.zeros((1, 2) + N[:-1] + (N[-1] // 2 + 1,), dtype=np.complex128)
    full[(slice(None), slice(None)) + np.ix_(*O.mode_index_lists(N, k))] = Y
    ref = np.fft.irfftn(full, s=N, axes=tuple(range(2, 2 + len(N))))
    assert O.rel_l2(O.inverse(Y, N, k), ref) < 1e-12


@settings(**SETTINGS)
@given(layer_shapes(), st.integers(0, 2 ** 31 - 1))
def test_slab_partials_sum_to_the_whole_for_every_divisor(shape, seed):
    N, k = shape
    x = np.random.default_rng(seed).standard_normal((1, 1) + N)
    whole = O.forward(x, k)
    for P in [p for p in range(1, N[0] + 1) if N[0] % p == 0]:
        nl = N[0] // P
        parts = sum(O.forward(x[:, :, p * nl:(p + 1) * nl], k, N_global=N, offsets=(p * nl,) + (0,) * (len(N) - 1))
                    for p in range(P))
        assert O.rel_l2(parts, whole) < 1e-12


@settings(**SETTINGS)
@given(layer_shapes(), st.integers(0, 2 ** 31 - 1))
def test_adjoint_identity_and_gradient_of_the_layer(shape, seed):
    torch = pytest.importorskip("torch")
    N, k = shape
    rng = np.random.default_rng(seed)
    B, Ci, Co = 1, 2, 2
    lists = O.mode_index_lists(N, k)
    K = tuple(len(l) for l in lists)
    M = math.prod(K)
    x = rng.standard_normal((B, Ci) + N)
    g = rng.standard_normal((B, Co) + N)
    W = (rng.standard_normal((Ci, Co, M)) + 1j * rng.standard_normal((Ci, Co, M))) / 2.0
    # <F x, Y> = <x, F^H Y>
    Yr = rng.standard_normal((B, Ci) + K) + 1j * rng.standard_normal((B, Ci) + K)
    lhs = np.sum(np.real(np.conj(O.forward(x, k)) * Yr))
    rhs = np.sum(x * O.inverse(Yr, N, k, doubling=False, normalise=False))
    assert abs(lhs - rhs) <= 1e-10 * max(1.0, abs(lhs))
    # backward == autograd through the library FFT
    y, Xhat = O.layer_forward(x, W, k)
    gx, gW = O.backward(g, Xhat, W.reshape((Ci, Co) + K), k)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W.reshape((Ci, Co) + K), dtype=torch.complex128, requires_grad=True)
    dims = tuple(range(2, 2 + len(N)))
    full = torch.fft.rfftn(xt, dim=dims)
    ix = torch.meshgrid(*[torch.as_tensor(l) for l in lists], indexing="ij")
    Xt = full[(slice(None), slice(None)) + tuple(ix)]
    letters = "pqrs"[:len(N)]
    Yt = torch.einsum(f"bi{letters},io{letters}->bo{letters}", Xt, Wt)
    pad = torch.zeros((B, Co) + N[:-1] + (N[-1] // 2 + 1,), dtype=torch.complex128)
    pad = pad.index_put(tuple([torch.arange(B)[:, None].reshape((B, 1) + (1,) * len(N)).expand((B, Co) + K),
                               torch.arange(Co).reshape((1, Co) + (1,) * len(N)).expand((B, Co) + K)] +
                              [t.expand((B, Co) + K) for t in ix]), Yt)
    yt = torch.fft.irfftn(pad, s=N, dim=dims)
    assert O.rel_l2(yt.detach().numpy(), y) < 1e-11
    (yt * torch.tensor(g)).sum().backward()
    assert O.rel_l2(xt.grad.numpy(), gx) < 1e-10
    # complex gradient in torch's convention dL/dRe + i dL/dIm, the one the ABI documents
    assert O.rel_l2(Wt.grad.numpy(), gW) < 1e-10
