"""The oracle at the benchmark's configurations, against numpy.fft (the paper's
own exactness experiment: FFT-then-truncate vs partial DFT, Section "Numerical
Exactness"), on the seeded synthetic inputs the GPU tests use."""
import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import inputs as I


def _fft_slice(x, kmax):
    N = x.shape[2:]
    full = np.fft.rfftn(x.astype(np.float64), axes=tuple(range(2, x.ndim)))
    return full[np.ix_(range(x.shape[0]), range(x.shape[1]), *O.mode_index_lists(N, kmax))]


@pytest.mark.parametrize("name,channels", [("cfg1_2d_64", None), ("cfg2_3d_64", 2), ("cfg3_4d_64", 1)])
def test_forward_matches_rfftn_slice_at_config_sizes(name, channels):
    w = I.WORKLOADS[name]
    x = I.make_field(w, channels)
    assert x.dtype == np.float32 and x.shape[2:] == w.N
    X = O.forward(x, w.kmax)
    assert X.shape[2:] == w.K
    assert O.rel_l2(X, _fft_slice(x, w.kmax)) < 1e-12


def test_sampled_literal_modes_at_config_size():
    # one mode = one prod(N)-term dot product (Eq. 5 as written), at cfg3's grid
    w = I.WORKLOADS["cfg3_4d_64"]
    x = I.make_field_channel(w, 0, 0)
    X = O.forward(x[None, None], w.kmax)[0, 0]
    lists = O.mode_index_lists(w.N, w.kmax)
    rng = np.random.default_rng(5)
    for _ in range(4):
        pos = tuple(int(rng.integers(0, len(s))) for s in lists)
        modes = [lists[j][pos[j]] for j in range(w.d)]
        v = O.forward_one_mode(x, w.N, modes)
        assert abs(v - X[pos]) <= 1e-10 * max(1.0, abs(v))


def test_input_generators_are_seeded_and_shaped():
    w = I.WORKLOADS["cfg2_3d_64"]
    a = I.make_field_channel(w, 1, 3)
    b = I.make_field_channel(w, 1, 3)
    assert np.array_equal(a, b)
    assert not np.array_equal(a, I.make_field_channel(w, 1, 4))
    assert abs(float(a.std()) - 1.0) < 0.05
    Wt = I.make_weights(w)
    assert Wt.shape == (16, 16, w.M) and Wt.dtype == np.complex64
    assert abs(float(Wt.real.var()) - 1.0 / 256) < 2e-4
    # smooth field: the retained low modes hold far more than their share of the energy
    X = np.fft.rfftn(a.astype(np.float64))
    tot = np.sum(np.abs(X) ** 2)
    low = np.sum(np.abs(X[np.ix_(*O.mode_index_lists(w.N, w.kmax))]) ** 2)
    assert low / tot > 0.25   # white noise would give ~0.05
    for name, wl in I.WORKLOADS.items():
        assert wl.M == O.num_modes(wl.N, wl.kmax)
