"""The DTST primitive proper on the GPU - complex fields, two-sided retained set on every dimension - through the
C ABI against the float64 oracle: forward, mixing, inverse, backward, virtual shards and a rank's block."""
import numpy as np
import pytest

from oracle import dtst_oracle as O

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _c64(rng, shape):
    return (rng.standard_normal(shape) + 1j * rng.standard_normal(shape)).astype(np.complex64)


CASES = [
    ("d1", 2, 2, 3, (16,), (5,)),
    ("d2_full_band", 1, 2, 2, (6, 8), (3, 4)),
    ("d3", 2, 3, 2, (16, 12, 24), (3, 2, 5)),
    ("d3_folded_mid", 1, 2, 2, (32, 64, 16), (8, 4, 3)),   # dims 0 and 1 on the folded tensor-core kernels
    ("d4", 1, 2, 1, (4, 6, 5, 8), (2, 1, 2, 3)),
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
@pytest.mark.parametrize("P", [1, 2])
def test_complex_layer_matches_the_oracle(case, P):
    from paper_2607_14394_b200 import Plan
    name, B, Ci, Co, N, k = case
    rng = np.random.default_rng(hash(name) % 1000)
    plan = Plan(N, k, B, Ci, Co, complex_fields=True, virtual_shards=P)
    lists = O.mode_index_lists_complex(N, k)
    for j in range(len(N)):
        assert plan.mode_indices(j) == lists[j].tolist()
    assert plan.K == tuple(2 * kk for kk in k)
    x, g = _c64(rng, (B, Ci) + N), _c64(rng, (B, Co) + N)
    W = (_c64(rng, (Ci, Co, plan.M)) / np.sqrt(Ci * Co)).astype(np.complex64)
    Xhat = plan.forward(_dev(x))
    Yhat = plan.spectral_mul(Xhat, _dev(W))
    y = plan.inverse(Yhat)
    gx, gW = plan.backward(_dev(g), Xhat, _dev(W))
    torch.cuda.synchronize()
    assert plan.status() == 0 and y.dtype == torch.complex64 and gx.dtype == torch.complex64
    y_ref, X_ref = O.layer_forward_complex(x, W, k)
    gx_ref, gW_ref = O.backward_complex(g, X_ref, W, k)
    errs = {"Xhat": O.rel_l2(Xhat.cpu().numpy(), X_ref), "y": O.rel_l2(y.cpu().numpy(), y_ref),
            "grad_x": O.rel_l2(gx.cpu().numpy(), gx_ref), "grad_W": O.rel_l2(gW.cpu().numpy(), gW_ref)}
    for n_, e in errs.items():
        assert e <= TOL, (name, P, n_, e, errs)


def test_complex_rank_block_and_wrong_entry_points():
    from paper_2607_14394_b200 import Plan, binding as Bn
    Ng, k, nl, off = (16, 12, 8), (3, 2, 4), (4, 12, 8), (8, 0, 0)
    rng = np.random.default_rng(5)
    x = _c64(rng, (1, 2) + Ng)
    blk = np.ascontiguousarray(x[:, :, 8:12])
    plan = Plan(nl, k, 1, 2, 2, N_global=Ng, offset=off, complex_fields=True)
    part = plan.forward(_dev(blk)).cpu().numpy()
    assert O.rel_l2(part, O.forward_complex(blk, k, N_global=Ng, offsets=off)) <= TOL
    Y = _c64(rng, part.shape)
    yb = plan.inverse(_dev(Y)).cpu().numpy()
    assert O.rel_l2(yb, O.inverse_complex(Y, Ng, k, n_local=nl, offsets=off)) <= TOL
    # the real-field entry points refuse a complex plan, and the other way round
    xr = torch.zeros((1, 2) + nl, device="cuda")
    out = torch.zeros((1, 2) + plan.K, dtype=torch.complex64, device="cuda")
    with pytest.raises(Bn.DtstError) as e:
        Bn.dtst_forward(plan.handle, xr, out)
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG
    real_plan = Plan((8, 8), (2, 2), 1, 1, 1)
    with pytest.raises(Bn.DtstError) as e:
        Bn.dtst_forward_complex(real_plan.handle, torch.zeros((1, 1, 8, 8), dtype=torch.complex64, device="cuda"),
                                torch.zeros((1, 1, 4, 2), dtype=torch.complex64, device="cuda"))
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG
