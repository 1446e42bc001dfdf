"""The whole block of Algorithm 1 on the GPU - GELU(W_bypass x + I(M(F(x), W))) and its backward pass, called
through the C ABI - against the float64 oracle on the same seeded inputs (rel-L2 <= 1e-5 per output tensor, every
plane on its own scale)."""
import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import inputs as I
from parity_checks import per_mode_excess, per_plane_excess

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _bypass_weights(w, seed=5):
    rng = np.random.default_rng(w.seed * 31 + seed)
    return (rng.standard_normal((w.C_out, w.C_in)) / np.sqrt(w.C_in)).astype(np.float32)


def run_block_and_check(w, path="auto", P=1, w_scale=1.0, epilogue="auto"):
    from paper_2607_14394_b200 import Plan
    x, W, g = I.make_field(w), I.make_weights(w) * np.float32(w_scale), I.make_upstream_grad(w)
    Wb = _bypass_weights(w)
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P, path=path)
    plan.set_block_epilogue(epilogue)
    xd, Wd, Wbd, gd = _dev(x), _dev(W), _dev(Wb), _dev(g)
    out, Xhat, z = plan.block_forward(xd, Wd, Wbd)
    out_nz, _, z_none = plan.block_forward(xd, Wd, Wbd, save_z=False)
    torch.cuda.synchronize()
    assert plan.status() == 0 and z_none is None
    assert torch.equal(out, out_nz)
    Wm = W.reshape((w.C_in, w.C_out) + w.K)
    out_ref, z_ref, X_ref = O.block_forward(x, Wm, Wb, w.kmax)
    errs = {"out": O.rel_l2(out.cpu().numpy(), out_ref), "z": O.rel_l2(z.cpu().numpy(), z_ref),
            "Xhat": O.rel_l2(Xhat.cpu().numpy(), X_ref)}
    fine = {"out/plane": per_plane_excess(out.cpu().numpy(), out_ref), "z/plane": per_plane_excess(z.cpu().numpy(), z_ref)}
    gx, gW, gWb = plan.block_backward(gd, xd, z, Xhat, Wd, Wbd)
    gx2, gW2, gWb2 = plan.block_backward(gd, xd, z, Xhat, Wd, Wbd)
    torch.cuda.synchronize()
    assert plan.status() == 0
    assert torch.equal(gx, gx2) and torch.equal(gWb, gWb2)           # fixed-order reduction: same bits
    gx_ref, gW_ref, gWb_ref = O.block_backward(g, x, z_ref, X_ref, Wm, Wb, w.kmax)
    errs["grad_x"] = O.rel_l2(gx.cpu().numpy(), gx_ref)
    errs["grad_W"] = O.rel_l2(gW.cpu().numpy().reshape(gW_ref.shape), gW_ref)
    errs["grad_W_bypass"] = O.rel_l2(gWb.cpu().numpy(), gWb_ref)
    fine["grad_x/plane"] = per_plane_excess(gx.cpu().numpy(), gx_ref)
    fine["grad_W/mode"] = per_mode_excess(gW.cpu().numpy().reshape(gW_ref.shape), gW_ref)
    for name, e in errs.items():
        assert e <= TOL, (w.name, path, P, name, e, errs)
    for name, e in fine.items():
        assert e <= 1.0, (w.name, path, P, name, e, fine)
    # the pieces one by one: only the bypass weight gradient, only the input gradient
    only_wb = torch.empty_like(gWb)
    from paper_2607_14394_b200 import binding as Bn
    scratch = torch.empty_like(z)
    Bn.dtst_block_backward(plan.handle, gd, xd, z, None, Wd, Wbd, scratch, None, None, only_wb)
    torch.cuda.synchronize()
    assert torch.equal(only_wb, gWb)
    plan.close()
    return errs


@pytest.mark.parametrize("name", ["cfg1_2d_64", "cfg2_3d_64", "cfg3_4d_64"])
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_block_benchmark_configs(name, path):
    # spectral weights scaled up so that the spectral term and the bypass term of z are of the same order
    run_block_and_check(I.WORKLOADS[name], path, w_scale=4.0)


BLOCK_EDGE = [
    ("c_odd", 2, 3, 2, (6, 8), (3, 5)),              # channel counts that are no multiple of 4, tiny grid
    ("c_wide", 1, 5, 7, (12, 20, 36), (3, 5, 7)),
    ("c_1", 1, 1, 1, (8, 16), (2, 4)),
    ("c_16_32", 1, 16, 32, (16, 32, 32), (4, 8, 8)),  # channel counts the tensor-core bypass kernel serves
    ("c_8_16_tail", 2, 8, 16, (10, 6, 44), (2, 3, 3)),  # grid points per channel not a multiple of the point tile
    ("d1", 3, 2, 2, (128,), (7,)),
]


@pytest.mark.parametrize("case", BLOCK_EDGE, ids=[c[0] for c in BLOCK_EDGE])
def test_block_edge_shapes(case):
    name, B, Ci, Co, N, k = case
    run_block_and_check(I.custom_workload(name, B, Ci, Co, N, k, field="grf" if len(N) > 1 else "iid", seed=13),
                        w_scale=4.0)


TENSOR_CASES = [
    ("t_16_16", 1, 16, 16, (16, 32, 32), (4, 8, 8)),
    ("t_8_16_tail", 2, 8, 16, (10, 6, 44), (2, 3, 3)),     # points per channel not a multiple of the 128-point tile
    ("t_32_32", 1, 32, 32, (8, 16, 32), (2, 4, 8)),
    ("t_16_32_many_tiles", 1, 16, 32, (64, 64, 32), (4, 8, 8)),   # more tiles than CTAs: the pipelines wrap around
]


@pytest.mark.parametrize("case", TENSOR_CASES, ids=[c[0] for c in TENSOR_CASES])
def test_block_epilogue_on_the_tensor_cores(case):
    """The bypass product as tcgen05.mma kind::tf32 with the accumulator in tensor memory, asked for explicitly,
    against the oracle; and the FFMA epilogue on the same inputs."""
    name, B, Ci, Co, N, k = case
    w = I.custom_workload(name, B, Ci, Co, N, k, field="grf", seed=17)
    run_block_and_check(w, w_scale=4.0, epilogue="tensor")
    run_block_and_check(w, w_scale=4.0, epilogue="ffma")


def test_block_epilogue_choice_is_validated():
    from paper_2607_14394_b200 import Plan, binding as Bn
    plan = Plan((8, 16), (2, 4), 1, 3, 5)
    with pytest.raises(Bn.DtstError) as e:
        plan.set_block_epilogue("tensor")           # channel counts the MMA tile does not fit
    assert e.value.status == Bn.DTST_ERR_UNSUPPORTED
    plan.set_block_epilogue("ffma")
    with pytest.raises(Bn.DtstError):
        Bn.dtst_plan_set_block_epilogue(plan.handle, 7)


def test_block_with_virtual_shards():
    run_block_and_check(I.custom_workload("blk_shards", 1, 4, 4, (16, 16, 32), (3, 4, 5), field="grf", seed=3), P=4,
                        w_scale=4.0)


def test_block_argument_errors():
    from paper_2607_14394_b200 import Plan, binding as Bn
    w = I.custom_workload("blk_err", 1, 2, 2, (8, 8), (2, 2))
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
    x = torch.zeros((1, 2, 8, 8), device="cuda")
    W = torch.zeros((2, 2, 8), dtype=torch.complex64, device="cuda")
    Wb = torch.zeros((2, 2), device="cuda")
    with pytest.raises(ValueError):
        plan.block_forward(x, W, torch.zeros((2, 3), device="cuda"))
    out, X, z = plan.block_forward(x, W, Wb)
    before = plan.launch_count()
    with pytest.raises(Bn.DtstError) as e:     # out aliasing x
        Bn.dtst_block_forward(plan.handle, x, W, Wb, x, X, None)
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG
    with pytest.raises(Bn.DtstError) as e:     # nothing asked for
        Bn.dtst_block_backward(plan.handle, x, x, z, X, W, Wb, out, None, None, None)
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG
    assert plan.launch_count() == before
