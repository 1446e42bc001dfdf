"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every
symbol the header declares, validates arguments, and its mode-index tables match
the oracle bit for bit."""
import ctypes
import os
import re

import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import binding as Bn
from paper_2607_14394_b200 import build as Bd
from paper_2607_14394_b200 import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    Bd.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "dtst.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dtst_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = Bn.lib()
    names = _declared_symbols()
    assert len(names) >= 18
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(Bn.EXPORTED)
    assert Bn.dtst_version() >= 100
    assert Bn.status_string(0) == "ok"
    assert "workspace" in Bn.status_string(Bn.DTST_ERR_WORKSPACE)


@pytest.mark.parametrize("name", list(I.WORKLOADS))
def test_mode_tables_match_oracle_bit_exact(name):
    w = I.WORKLOADS[name]
    h = Bn.dtst_plan_create(w.d, w.N, w.kmax, w.B, w.C_in, w.C_out)
    try:
        M, K = Bn.dtst_plan_num_modes(h, w.d)
        assert M == O.num_modes(w.N, w.kmax) == w.M
        lists = O.mode_index_lists(w.N, w.kmax)
        assert K == tuple(len(s) for s in lists)
        for j in range(w.d):
            assert Bn.dtst_plan_mode_indices(h, j, K[j]) == lists[j].tolist()
        assert Bn.dtst_plan_workspace_bytes(h) >= 256
    finally:
        Bn.dtst_plan_destroy(h)


def test_edge_mode_tables():
    for N, k in [((7,), (4,)), ((8,), (5,)), ((6, 8), (3, 5)), ((5, 6), (1, 1))]:
        h = Bn.dtst_plan_create(len(N), N, k, 1, 1, 1)
        M, K = Bn.dtst_plan_num_modes(h, len(N))
        lists = O.mode_index_lists(N, k)
        for j in range(len(N)):
            assert Bn.dtst_plan_mode_indices(h, j, K[j]) == lists[j].tolist()
        Bn.dtst_plan_destroy(h)


@pytest.mark.parametrize("d,N,k,B,Ci,Co", [
    (0, (8,), (2,), 1, 1, 1),            # d out of range
    (7, (8,) * 7, (2,) * 7, 1, 1, 1),
    (2, (8, 8), (5, 2), 1, 1, 1),        # 2k > N on a two-sided dim
    (2, (8, 8), (2, 6), 1, 1, 1),        # beyond Nyquist on the one-sided dim
    (2, (8, 8), (0, 2), 1, 1, 1),        # k < 1
    (2, (8, 0), (2, 1), 1, 1, 1),        # empty grid
    (2, (8, 8), (2, 2), 0, 1, 1),        # empty batch
    (2, (8, 8), (2, 2), 1, 0, 1),
    (2, (8, 8), (2, 2), 1, 1, -3),
])
def test_plan_create_rejects_bad_arguments(d, N, k, B, Ci, Co):
    with pytest.raises(Bn.DtstError) as e:
        Bn.dtst_plan_create(d, N, k, B, Ci, Co)
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG


def test_local_plan_validation_and_shards():
    with pytest.raises(Bn.DtstError):
        Bn.dtst_plan_create_local(2, (16, 8), (8, 8), (12, 0), (2, 2), 1, 1, 1)   # block sticks out
    h = Bn.dtst_plan_create_local(2, (16, 8), (4, 8), (12, 0), (2, 2), 1, 1, 1)
    with pytest.raises(Bn.DtstError):
        Bn.dtst_plan_set_virtual_shards(h, 3)       # 3 does not divide 4
    base = Bn.dtst_plan_workspace_bytes(h)
    Bn.dtst_plan_set_virtual_shards(h, 2)
    assert Bn.dtst_plan_workspace_bytes(h) > base   # partial spectra need room
    with pytest.raises(Bn.DtstError):
        Bn.dtst_plan_set_kernel_path(h, 7)
    Bn.dtst_plan_destroy(h)


def test_null_handles_are_errors_not_crashes():
    lib = Bn.lib()
    null = ctypes.c_void_p(0)
    assert lib.dtst_plan_destroy(null) == Bn.DTST_ERR_INVALID_ARG
    assert lib.dtst_forward(null, null, null, null) == Bn.DTST_ERR_INVALID_ARG
    assert lib.dtst_plan_create(None, 1, None, None, 1, 1, 1) == Bn.DTST_ERR_INVALID_ARG
    h = Bn.dtst_plan_create(1, (8,), (2,), 1, 1, 1)
    # no workspace yet -> compute calls refuse before touching any pointer
    assert lib.dtst_forward(h, null, null, null) == Bn.DTST_ERR_WORKSPACE
    assert lib.dtst_inverse(h, null, null, null) == Bn.DTST_ERR_WORKSPACE
    assert lib.dtst_spectral_mul(h, null, null, null, null) == Bn.DTST_ERR_INVALID_ARG
    assert lib.dtst_plan_set_workspace(h, ctypes.c_void_p(128), 1 << 20) == Bn.DTST_ERR_INVALID_ARG  # misaligned
    Bn.dtst_plan_destroy(h)


def test_host_io_argument_checks_need_no_gpu():
    import ctypes
    lib = Bn.lib()
    n = ctypes.c_size_t()
    assert lib.dtst_plan_host_io_bytes(None, ctypes.byref(n)) == Bn.DTST_ERR_INVALID_ARG
    h = Bn.dtst_plan_create(2, (32, 64), (4, 8), 1, 2, 3)
    try:
        assert lib.dtst_plan_host_io_bytes(h, ctypes.byref(n)) == Bn.DTST_OK
        grid_in, grid_out, M = 2 * 32 * 64 * 4, 3 * 32 * 64 * 4, 8 * 8
        want = 2 * grid_in + 2 * grid_out + (2 + 3 + 6) * M * 8
        assert want <= n.value <= want + 7 * 256       # seven regions, each rounded up to 256 bytes
        # not enabled: a step is refused, nothing runs
        assert lib.dtst_step_host(h, None, None, None, None, None, None) == Bn.DTST_ERR_INVALID_ARG
        assert lib.dtst_host_io_wait(h) == Bn.DTST_ERR_INVALID_ARG
        assert lib.dtst_plan_enable_host_io(h, ctypes.c_void_p(4), n.value) == Bn.DTST_ERR_INVALID_ARG   # misaligned
        assert lib.dtst_plan_enable_host_io(h, None, 0) == Bn.DTST_OK                                  # off: no-op
    finally:
        Bn.dtst_plan_destroy(h)
