"""The C ABI from plain C: a gcc-built driver (tests/c_driver/dtst_c_driver.c, no Python, no C++) runs forward ->
spectral_mul -> inverse on seeded inputs written to files; its outputs are compared with the float64 oracle."""
import subprocess

import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import build as B
from paper_2607_14394_b200 import inputs as I

TOL = 1e-5


def test_c_driver_builds_and_rejects_bad_usage():
    exe = B.build_c_driver()
    res = subprocess.run([exe], capture_output=True, text=True)
    assert res.returncode == 64
    res = subprocess.run([exe, "9"], capture_output=True, text=True)
    assert res.returncode == 64 and "usage" in res.stderr


@pytest.mark.gpu
@pytest.mark.parametrize("N,k", [((32, 32, 64), (4, 4, 8)), ((10, 6, 12), (2, 3, 3)), ((64, 64), (8, 8))])
def test_c_driver_matches_oracle(tmp_path, N, k):
    exe = B.build_c_driver()
    w = I.custom_workload("c_driver", 2, 3, 2, N, k, field="grf", seed=71)
    x, W = I.make_field(w), I.make_weights(w)
    fx, fW, fX, fy = (str(tmp_path / n) for n in ("x.bin", "W.bin", "Xhat.bin", "y.bin"))
    x.astype(np.float32).tofile(fx)
    W.astype(np.complex64).tofile(fW)
    args = [exe, str(w.d)] + [str(n) for n in N] + [str(v) for v in k] + [str(w.B), str(w.C_in), str(w.C_out),
                                                                           fx, fW, fX, fy]
    res = subprocess.run(args, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "kernel launches" in res.stdout and "kernel launches: 0" not in res.stdout
    Xhat = np.fromfile(fX, dtype=np.complex64).reshape((w.B, w.C_in) + w.K)
    y = np.fromfile(fy, dtype=np.float32).reshape((w.B, w.C_out) + tuple(N))
    y_ref, X_ref = O.layer_forward(x, W, w.kmax)
    assert O.rel_l2(Xhat, X_ref) <= TOL
    assert O.rel_l2(y, y_ref) <= TOL
