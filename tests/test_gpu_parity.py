"""GPU parity: the CUDA path, called through the C ABI, against the float64 oracle
on the same seeded inputs.  Bar: rel-L2 <= 1e-5 over each whole output tensor
(complex as two reals, compared in float64) and bit-exact mode-index tables."""
import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import inputs as I
from parity_checks import per_mode_excess, per_plane_excess

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


def _plan(w, path="auto", P=1, **kw):
    from paper_2607_14394_b200 import Plan
    return Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P, path=path, **kw)


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def run_layer_and_check(w, path="auto", P=1, check_backward=True, tol=TOL, fine_scale=1.0, **plan_kw):
    x = I.make_field(w)
    W = I.make_weights(w)
    g = I.make_upstream_grad(w)
    plan = _plan(w, path, P, **plan_kw)
    lists = O.mode_index_lists(w.N, w.kmax)
    for j in range(w.d):
        assert plan.mode_indices(j) == lists[j].tolist()
    xd, Wd, gd = _dev(x), _dev(W), _dev(g)
    Xhat = plan.forward(xd)
    Yhat = plan.spectral_mul(Xhat, Wd)
    y = plan.inverse(Yhat)
    torch.cuda.synchronize()
    assert plan.status() == 0

    X_ref = O.forward(x, w.kmax)
    Wm = W.reshape((w.C_in, w.C_out) + w.K)
    Y_ref = O.spectral_mul(X_ref, Wm)
    y_ref = O.inverse(Y_ref, w.N, w.kmax)
    errs = {
        "Xhat": O.rel_l2(Xhat.cpu().numpy(), X_ref),
        "Yhat": O.rel_l2(Yhat.cpu().numpy(), Y_ref),
        "y": O.rel_l2(y.cpu().numpy(), y_ref),
    }
    # every retained mode and every plane on its own scale (multiples of the per-mode / per-plane bars)
    fine = {
        "Xhat/mode": per_mode_excess(Xhat.cpu().numpy(), X_ref),
        "Yhat/mode": per_mode_excess(Yhat.cpu().numpy(), Y_ref),
        "y/plane": per_plane_excess(y.cpu().numpy(), y_ref),
    }
    if check_backward:
        gx, gW = plan.backward(gd, Xhat, Wd)
        torch.cuda.synchronize()
        gx_ref, gW_ref = O.backward(g, X_ref, Wm, w.kmax)
        errs["grad_x"] = O.rel_l2(gx.cpu().numpy(), gx_ref)
        errs["grad_W"] = O.rel_l2(gW.cpu().numpy().reshape(gW_ref.shape), gW_ref)
        fine["grad_W/mode"] = per_mode_excess(gW.cpu().numpy().reshape(gW_ref.shape), gW_ref)
        fine["grad_x/plane"] = per_plane_excess(gx.cpu().numpy(), gx_ref)
    for name, e in errs.items():
        assert e <= tol, (w.name, path, P, name, e, errs)
    for name, e in fine.items():     # fine_scale: the per-mode / per-plane bars scaled with a looser tolerance
        assert e <= fine_scale, (w.name, path, P, name, e, fine)
    plan.close()
    return errs


# ------------------------------------------------------------------ the benchmark's small configs, in full
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_cfg1_2d(path):
    run_layer_and_check(I.WORKLOADS["cfg1_2d_64"], path)


@pytest.mark.parametrize("path", ["auto", "generic"])
def test_cfg2_3d(path):
    run_layer_and_check(I.WORKLOADS["cfg2_3d_64"], path)


@pytest.mark.parametrize("path", ["auto", "generic"])
def test_cfg3_4d(path):
    run_layer_and_check(I.WORKLOADS["cfg3_4d_64"], path)


# ------------------------------------------------------------------ edge shapes (generic path serves all of them)
EDGE = [
    # name, B, Ci, Co, N, kmax
    ("d1_odd", 2, 3, 2, (7,), (4,)),
    ("d1_nyquist", 1, 2, 2, (8,), (5,)),
    ("d2_full_band", 1, 2, 3, (6, 8), (3, 5)),       # 2k = N and Nyquist
    ("d2_k1", 2, 1, 1, (5, 6), (1, 1)),
    ("d3_ragged", 1, 3, 2, (10, 6, 12), (2, 3, 3)),
    ("d4_small", 1, 2, 2, (4, 6, 5, 8), (2, 1, 2, 3)),
    ("d5", 1, 2, 1, (4, 3, 6, 4, 8), (2, 1, 2, 2, 3)),            # more dimensions than the benchmark uses
    ("d6", 1, 1, 2, (2, 4, 3, 4, 2, 8), (1, 2, 1, 1, 1, 2)),
    ("d5_fused_tail", 1, 1, 1, (2, 2, 32, 64, 32), (1, 1, 4, 8, 4)),   # d = 5 with plane + folded kernels inside
    ("big_batch", 6, 2, 3, (8, 16), (2, 4)),          # B > the mixing kernels' batch tile
    ("tail_rows", 1, 5, 7, (12, 20, 36), (3, 5, 7)),  # nothing a multiple of a tile
    ("wide_last", 1, 2, 2, (8, 8, 520), (2, 3, 9)),
    # shapes served by the one-dimension streaming kernels: N3 a multiple of 32, ragged row counts
    ("row_32_k16", 1, 3, 2, (5, 32), (2, 16)),
    ("row_96_odd_k", 2, 1, 3, (3, 7, 96), (1, 3, 5)),
    ("row_160", 1, 2, 1, (6, 160), (3, 9)),
    ("row_256", 1, 1, 2, (4, 6, 256), (2, 3, 16)),
    ("row_d1", 3, 2, 2, (128,), (7,)),
    ("row_k1", 1, 2, 2, (9, 64), (4, 1)),
    # middle dimensions on the tensor-core kernels (N % 32 == 0, inner extent a multiple of 4): k = 4 / 8 / 12 / 16,
    # N not a power of two, column tiles that end inside a task, a single column tile
    ("mid_mma_k4", 1, 2, 2, (32, 32, 64), (4, 4, 2)),
    ("mid_mma_n96_k12", 1, 2, 1, (96, 64, 32), (12, 8, 6)),
    ("mid_mma_tail", 1, 2, 2, (64, 32, 32), (16, 4, 5)),
    ("mid_mma_thin", 2, 1, 2, (32, 64, 32), (8, 8, 4)),
]


@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_edge_shapes(case, path):
    name, B, Ci, Co, N, k = case
    run_layer_and_check(I.custom_workload(name, B, Ci, Co, N, k, seed=11), path)


# ------------------------------------------------------------------ a seeded sweep of shapes nobody picked by hand
def _random_cases(count, seed):
    """Seeded draw of (B, C_in, C_out, N, kmax, P): d = 1..4, extents that mix multiples of 32 / 16 / 4 with odd
    numbers where the ABI allows them, retained counts from 1 up to the full band, a virtual-shard count that
    divides N_0.  Sizes stay small enough for the oracle to take a fraction of a second each."""
    rng = np.random.default_rng(seed)
    last_choices = [4, 8, 12, 20, 32, 36, 64, 96, 128]          # the contiguous extent must be a multiple of 4
    mid_choices = [3, 4, 5, 6, 8, 9, 12, 16, 24, 32, 33, 64]
    cases = []
    while len(cases) < count:
        d = int(rng.integers(1, 5))
        N = [int(rng.choice(mid_choices)) for _ in range(d - 1)] + [int(rng.choice(last_choices))]
        if np.prod(N) > 300_000:
            continue
        k = []
        for j, n in enumerate(N):
            hi = n // 2 if j < d - 1 else n // 2 + 1
            k.append(int(rng.integers(1, max(1, min(hi, 16)) + 1)))
        B, Ci, Co = int(rng.integers(1, 4)), int(rng.integers(1, 5)), int(rng.integers(1, 5))
        divs = [p for p in (1, 2, 3, 4, 8) if N[0] % p == 0]
        P = int(rng.choice(divs))
        cases.append((B, Ci, Co, tuple(N), tuple(k), P))
    return cases


RANDOM_CASES = _random_cases(28, seed=20260714)


@pytest.mark.parametrize("case", RANDOM_CASES, ids=[f"r{i}_" + "x".join(map(str, c[3])) for i, c in enumerate(RANDOM_CASES)])
def test_random_shapes(case):
    B, Ci, Co, N, k, P = case
    w = I.custom_workload("random", B, Ci, Co, N, k, field="grf" if len(N) > 1 else "iid", seed=sum(N) + 7 * P)
    run_layer_and_check(w, "auto", P=P)


# ------------------------------------------------------------------ virtual shards (Eq. 6-7 on one GPU)
@pytest.mark.parametrize("N,k,P", [((16, 8, 12), (3, 2, 4), 4), ((16, 8, 12), (3, 2, 4), 16),
                                   ((64, 64), (8, 8), 8), ((8,), (3,), 2),
                                   ((64, 32, 32, 16), (8, 4, 4, 4), 8),
                                   # slabs of whole 8-row steps: the tensor-core slab contraction, with column tails
                                   ((128, 64, 32), (16, 16, 4), 8), ((96, 32, 36), (12, 4, 9), 3),
                                   ((64, 128), (16, 12), 8)])
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_virtual_shards_match_oracle_and_unsharded(N, k, P, path):
    w = I.custom_workload("shards", 2, 2, 3, N, k, field="grf", seed=23)
    run_layer_and_check(w, path, P=P)
    x = _dev(I.make_field(w))
    a = _plan(w, path, 1).forward(x)
    b = _plan(w, path, P).forward(x)
    assert O.rel_l2(b.cpu().numpy(), a.cpu().numpy()) <= TOL
    # and the slab partial sums agree with the oracle's sharded statement
    ref = O.forward_sharded(I.make_field(w), w.kmax, P)
    assert O.rel_l2(b.cpu().numpy(), ref) <= TOL


# ------------------------------------------------------------------ a rank's block with global offsets (Eq. 18)
@pytest.mark.parametrize("Ng,k,nl,off", [((16, 12, 8), (3, 2, 4), (4, 6, 8), (8, 6, 0)),
                                         ((32, 24, 32), (4, 8, 4), (8, 12, 32), (16, 12, 0))])
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_local_block_plan_gives_partial_spectrum_and_block_inverse(path, Ng, k, nl, off):
    from paper_2607_14394_b200 import Plan
    w = I.custom_workload("local", 1, 2, 2, Ng, k, seed=31)
    x = I.make_field(w)
    sl = tuple(slice(o, o + n) for o, n in zip(off, nl))
    blk = np.ascontiguousarray(x[(slice(None), slice(None)) + sl])
    plan = Plan(nl, k, 1, 2, 2, N_global=Ng, offset=off, path=path)
    part = plan.forward(_dev(blk)).cpu().numpy()
    ref = O.forward(blk, k, N_global=Ng, offsets=off)
    assert O.rel_l2(part, ref) <= TOL
    Y = (np.random.default_rng(3).standard_normal(ref.shape) + 1j * np.random.default_rng(4).standard_normal(ref.shape))
    yb = plan.inverse(_dev(Y.astype(np.complex64))).cpu().numpy()
    yref = O.inverse(Y.astype(np.complex64), Ng, k, n_local=nl, offsets=off)
    assert O.rel_l2(yb, yref) <= TOL
    # and the block's backward pass against the oracle's block statement
    Wn = I.make_weights(w)
    g = np.random.default_rng(9).standard_normal((1, 2) + tuple(nl)).astype(np.float32)
    Xs = _dev(part.astype(np.complex64))
    gx, gW = plan.backward(_dev(g), Xs, _dev(Wn))
    gx_ref, gW_ref = O.backward(g, part.astype(np.complex64), Wn.reshape((2, 2) + ref.shape[2:]), k, N_global=Ng,
                                offsets=off)
    assert O.rel_l2(gx.cpu().numpy(), gx_ref) <= TOL
    assert O.rel_l2(gW.cpu().numpy().reshape(gW_ref.shape), gW_ref) <= TOL


# ------------------------------------------------------------------ run-to-run determinism and buffer discipline
@pytest.mark.parametrize("path", ["auto", "generic"])
def test_bitwise_reproducible_and_no_out_of_bounds_writes(path):
    w = I.custom_workload("repro", 2, 3, 3, (16, 12, 24), (3, 2, 5), seed=5)
    from paper_2607_14394_b200 import binding as Bn
    plan = _plan(w, path, P=4, allocate_workspace=False)
    nbytes = plan.workspace_bytes()
    guard = 4096
    ws = torch.full((nbytes + 2 * guard,), 0xA5, dtype=torch.uint8, device="cuda")
    Bn.dtst_plan_set_workspace(plan.handle, ws[guard:guard + nbytes])
    x, Wd, g = _dev(I.make_field(w)), _dev(I.make_weights(w)), _dev(I.make_upstream_grad(w))

    def padded(shape, dtype):
        n = int(np.prod(shape))
        pad = 64
        buf = torch.full((n + 2 * pad,), complex("nan+nanj") if dtype.is_complex else float("nan"),
                         dtype=dtype, device="cuda")
        return buf, buf[pad:pad + n].view(shape), pad

    outs = []
    for _ in range(2):
        Xb, X, pad = padded((w.B, w.C_in) + w.K, torch.complex64)
        Yb, Y, _ = padded((w.B, w.C_out) + w.K, torch.complex64)
        yb, y, _ = padded((w.B, w.C_out) + w.N, torch.float32)
        gxb, gx, _ = padded((w.B, w.C_in) + w.N, torch.float32)
        gWb, gW, _ = padded((w.C_in, w.C_out, w.M), torch.complex64)
        plan.forward(x, X)
        plan.spectral_mul(X, Wd, Y)
        plan.inverse(Y, y)
        plan.backward(g, X, Wd, gx, gW)
        torch.cuda.synchronize()
        for buf, view in ((Xb, X), (Yb, Y), (yb, y), (gxb, gx), (gWb, gW)):
            flat = torch.view_as_real(buf) if buf.is_complex() else buf
            assert torch.isnan(flat[:pad]).all() and torch.isnan(flat[-pad:]).all()
            assert not torch.isnan(torch.view_as_real(view) if view.is_complex() else view).any()
        outs.append([t.clone() for t in (X, Y, y, gx, gW)])
    for a, b in zip(*outs):
        assert torch.equal(torch.view_as_real(a) if a.is_complex() else a,
                           torch.view_as_real(b) if b.is_complex() else b)
    assert (ws[:guard] == 0xA5).all() and (ws[guard + nbytes:] == 0xA5).all()


def test_argument_errors_on_device():
    from paper_2607_14394_b200 import binding as Bn
    w = I.custom_workload("err", 1, 2, 2, (8, 8), (2, 2))
    plan = _plan(w)
    x = torch.zeros((1, 2, 8, 8), device="cuda")
    X = torch.zeros((1, 2, 4, 2), dtype=torch.complex64, device="cuda")
    lib = Bn.lib()
    import ctypes
    st = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.dtst_forward(plan.handle, ctypes.c_void_p(x.data_ptr() + 4), ctypes.c_void_p(X.data_ptr()), st) \
        == Bn.DTST_ERR_INVALID_ARG
    assert lib.dtst_spectral_mul(plan.handle, ctypes.c_void_p(X.data_ptr()), ctypes.c_void_p(X.data_ptr()),
                                 ctypes.c_void_p(X.data_ptr()), st) == Bn.DTST_ERR_INVALID_ARG   # aliasing
    assert lib.dtst_backward(plan.handle, ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(X.data_ptr()),
                             ctypes.c_void_p(X.data_ptr()), None, None, st) == Bn.DTST_ERR_INVALID_ARG
    # the saved spectrum is read for grad_W only: it may be missing when grad_W is not asked for ...
    Wt = torch.zeros((2, 2, 8), dtype=torch.complex64, device="cuda")
    gxt = torch.zeros_like(x)
    assert lib.dtst_backward(plan.handle, ctypes.c_void_p(x.data_ptr()), None, ctypes.c_void_p(Wt.data_ptr()),
                             ctypes.c_void_p(gxt.data_ptr()), None, st) == Bn.DTST_OK
    # ... and is required when it is
    assert lib.dtst_backward(plan.handle, ctypes.c_void_p(x.data_ptr()), None, ctypes.c_void_p(Wt.data_ptr()),
                             ctypes.c_void_p(gxt.data_ptr()), ctypes.c_void_p(Wt.data_ptr()), st) \
        == Bn.DTST_ERR_INVALID_ARG
    torch.cuda.synchronize()
    launched = plan.launch_count()
    # tensors of the wrong size never reach the kernels
    with pytest.raises(ValueError):
        plan.forward(torch.zeros((1, 2, 8, 4), device="cuda"))
    with pytest.raises(ValueError):
        plan.forward(x, out=torch.zeros((1, 2, 4, 1), dtype=torch.complex64, device="cuda"))
    with pytest.raises(ValueError):
        plan.spectral_mul(X, torch.zeros((2, 2, 4), dtype=torch.complex64, device="cuda"))
    with pytest.raises(ValueError):
        plan.inverse(X, out=torch.zeros((1, 2, 8, 7), device="cuda"))
    with pytest.raises(ValueError):
        plan.backward(x, X, Wt, grad_x=torch.zeros((1, 1, 8, 8), device="cuda"))
    with pytest.raises(ValueError):
        plan.spectral_mul_modes(X, Wt, 4, 8)
    assert plan.launch_count() == launched
    small = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(Bn.DtstError) as e:
        Bn.dtst_plan_set_workspace(plan.handle, small)
    assert e.value.status == Bn.DTST_ERR_WORKSPACE
    with pytest.raises(ValueError):
        plan.forward(x.cpu())
    assert plan.status() == 0
    before = plan.launch_count()
    plan.forward(x)
    assert plan.launch_count() > before


@pytest.mark.parametrize("which", ["plane", "plane_with_third_dimension"])
def test_bounded_wait_runs_out_and_is_reported_once(which):
    """The failure-reporting path of the streaming kernels, made to happen on the host's request: the forward
    plane kernel's producer stops feeding its ring after one fill, the consumers' bounded waits run out (and, in
    the kernel that also contracts the third dimension, the accumulator warps' waits for their batches), the
    kernel returns normally, dtst_plan_status reports the timeout once and clears it, and the next ordinary call
    is correct.  Nothing faults and no wait is unbounded."""
    from paper_2607_14394_b200 import binding as Bn
    w = I.WORKLOADS["cfg1_2d_64"] if which == "plane" else \
        I.custom_workload("colfuse_timeout", 1, 2, 2, (32, 128, 64), (16, 16, 8), field="iid", seed=5)
    plan = _plan(w, column_contraction=1)
    assert plan.kernel_path == "fused"
    x = _dev(I.make_field(w))
    ref = plan.forward(x).clone()
    torch.cuda.synchronize()
    assert plan.status() == Bn.DTST_OK
    plan.debug_ring_fault(1, poll_limit=1024)
    junk = plan.forward(x)
    assert plan.status() == Bn.DTST_ERR_DEVICE_TIMEOUT
    assert plan.status() == Bn.DTST_OK                       # reported once, then cleared
    plan.debug_ring_fault(-1)
    again = plan.forward(x)
    torch.cuda.synchronize()
    assert plan.status() == Bn.DTST_OK
    assert torch.equal(torch.view_as_real(again), torch.view_as_real(ref))
    assert O.rel_l2(again.cpu().numpy(), O.forward(I.make_field(w), w.kmax)) <= TOL
    del junk


def test_in_kernel_column_expansion_gives_the_same_bits():
    """The optional inverse-type kernel that expands dimension d-3 on a helper warp inside the plane kernel
    (flow control through per-column counters in global memory, a ring of columns consumed from L2) does the
    same arithmetic as the separate launch: same bits, for rings smaller and larger than the column count, and
    against the oracle."""
    from paper_2607_14394_b200 import Plan, binding as Bn
    w = I.WORKLOADS["cfg3_4d_64"]
    Wd, g = _dev(I.make_weights(w)), _dev(I.make_upstream_grad(w))
    x = _dev(I.make_field(w))
    ref_plan = _plan(w)
    Xhat = ref_plan.forward(x)
    Yhat = ref_plan.spectral_mul(Xhat, Wd)
    y_ref = ref_plan.inverse(Yhat)
    gx_ref, gW_ref = ref_plan.backward(g, Xhat, Wd)
    torch.cuda.synchronize()
    launches_ref = ref_plan.launch_count()
    for ring in (3, 16, 10_000):
        plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, column_expansion=ring)
        y = plan.inverse(Yhat)
        y2 = plan.inverse(Yhat)                       # the counters start every launch from zero
        gx, gW = plan.backward(g, Xhat, Wd)
        torch.cuda.synchronize()
        assert plan.status() == 0
        assert torch.equal(y, y_ref) and torch.equal(y2, y_ref) and torch.equal(gx, gx_ref)
        assert torch.equal(torch.view_as_real(gW), torch.view_as_real(gW_ref))
        plan.close()
    y_or = O.inverse(O.spectral_mul(O.forward(I.make_field(w), w.kmax), I.make_weights(w).reshape((w.C_in, w.C_out) + w.K)),
                     w.N, w.kmax)
    assert O.rel_l2(y_ref.cpu().numpy(), y_or) <= TOL
    # shapes without such a kernel say so
    w2 = I.custom_workload("nocolexp", 1, 2, 2, (16, 24, 40), (3, 5, 6))
    p2 = _plan(w2)
    with pytest.raises(Bn.DtstError) as e:
        Bn.dtst_plan_set_column_expansion(p2.handle, 8)
    assert e.value.status == Bn.DTST_ERR_UNSUPPORTED


# ------------------------------------------------------------------ more plane shapes than the benchmark's three
PLANE_SHAPES = [
    # name, B, Ci, Co, N, kmax: (N3, k3, N2, k2) of the last two dimensions is a shape the plane kernels exist for
    ("p_64_8_128_8", 1, 2, 2, (32, 128, 64), (4, 8, 8)),
    ("p_32_8_64_8", 1, 2, 3, (32, 32, 64, 32), (4, 8, 8, 8)),
    ("p_32_8_128_16", 1, 1, 2, (64, 128, 32), (8, 16, 8)),
    ("p_32_8_128_8", 2, 1, 1, (32, 128, 32), (16, 8, 8)),
    ("p_64_4_64_8", 1, 2, 2, (32, 64, 64), (12, 8, 4)),
    ("p_64_8_64_8_d3", 1, 2, 2, (64, 64, 64), (8, 8, 8)),
    # the paper's own layer shape in small: modes (8, 8, 8, 16) with 16 one-sided modes on a time axis of 32
    ("p_32_16_64_8_paper", 1, 2, 2, (32, 32, 64, 32), (8, 8, 8, 16)),
]


@pytest.mark.parametrize("case", PLANE_SHAPES, ids=[c[0] for c in PLANE_SHAPES])
def test_more_plane_shapes_run_fused_and_match_the_oracle(case):
    name, B, Ci, Co, N, k = case
    w = I.custom_workload(name, B, Ci, Co, N, k, field="grf", seed=29)
    plan = _plan(w)
    assert plan.kernel_path == "fused"
    plan.require_fast_path()            # every stage on a streaming kernel, or this raises
    plan.close()
    run_layer_and_check(w, "auto")
    run_layer_and_check(w, "auto", P=4)


# ------------------------------------------------------------------ contiguous extents that are no multiple of 32
ANY_EXTENT = [
    # name, B, Ci, Co, N, kmax, every stage streaming?
    # the paper's own grid in small: a time axis of 30 points with all 16 one-sided modes (the Nyquist mode included)
    ("g_paper_t30", 1, 2, 2, (16, 16, 32, 30), (4, 8, 8, 16), True),
    ("g_100", 1, 2, 3, (32, 32, 100), (8, 8, 12), True),
    ("g_odd_45", 2, 1, 2, (16, 32, 45), (4, 4, 12), True),           # odd extent: the middle sample has no partner
    ("g_odd_7_ragged", 1, 3, 1, (5, 7, 7), (2, 3, 4), False),        # 105 rows: a ragged last task, k3 = N3/2 + 1
    ("g_k3_20", 1, 2, 2, (32, 96), (8, 20), True),                   # three frequency tiles
    ("g_k3_32_odd_rows", 1, 1, 1, (9, 330), (4, 32), False),         # four frequency tiles, 9 rows
    ("g_k3_odd", 1, 2, 2, (32, 50), (8, 9), False),                  # odd mode count: 8-byte stores
    ("g_1d", 2, 3, 2, (90,), (17,), True),
    ("g_512", 1, 2, 2, (8, 512), (4, 16), True),                     # longer than the tensor-map kernels take
    ("g_421", 1, 3, 2, (45, 421), (12, 12), True),                   # long odd rows (8-row tasks), 135 rows: ragged
    # the second-last dimension inside the kernel: 24 and 32 modes (two mode tiles), 8 modes (half a tile), few
    # frequencies (two column tiles), 16-row tasks, and more planes than warps on the GPU (the ring crosses planes)
    ("g_plane_k2_12", 1, 2, 2, (16, 64, 60), (4, 12, 16), True),
    ("g_plane_k2_16_k3_6", 1, 1, 2, (16, 32, 44), (8, 16, 6), False),
    ("g_plane_k2_4", 2, 1, 1, (8, 96, 30), (4, 4, 11), False),
    ("g_plane_200", 1, 2, 1, (8, 48, 200), (4, 8, 16), True),
    ("g_plane_many", 2, 4, 4, (256, 32, 30), (8, 8, 16), True),
]


# ------------------------------------------------------------------ middle dimensions with any extent and mode count
ANY_MIDDLE = [
    # name, B, Ci, Co, N, kmax: mode counts the double-folded kernels are not built for, odd extents, odd inner extents
    ("m_k6", 1, 2, 2, (32, 64, 64), (6, 6, 8)),
    ("m_k10_k20", 1, 2, 1, (64, 64, 64), (10, 20, 16)),
    ("m_k32", 1, 1, 2, (64, 96, 32), (32, 5, 8)),
    ("m_odd_extents", 2, 1, 1, (45, 27, 64), (7, 13, 16)),
    ("m_odd_inner", 1, 2, 2, (40, 36, 50), (9, 3, 9)),          # k3 = 9: 8-byte copies
    ("m_2d_k24", 1, 3, 2, (100, 64), (24, 12)),
    ("m_4d", 1, 1, 2, (20, 24, 28, 32), (5, 6, 7, 8)),
    ("m_k1", 1, 2, 2, (6, 10, 32), (1, 2, 4)),
]


@pytest.mark.parametrize("case", ANY_MIDDLE, ids=[c[0] for c in ANY_MIDDLE])
def test_any_middle_extent_and_mode_count_runs_on_folded_kernels(case):
    name, B, Ci, Co, N, k = case
    w = I.custom_workload(name, B, Ci, Co, N, k, field="grf", seed=37)
    plan = _plan(w)
    plan.require_fast_path()            # every stage on a streaming kernel, or this raises
    plan.close()
    run_layer_and_check(w, "auto")
    if N[0] % 4 == 0:
        # virtual shards along dimension 0: its rows carry their global phases in the same folded kernels
        plan = _plan(w, P=4)
        plan.require_fast_path()
        plan.close()
        run_layer_and_check(w, "auto", P=4)


# ------------------------------------------------------------------ long contiguous extents (chunked row kernels)
LONG_ROWS = [
    # name, B, Ci, Co, N, kmax
    ("l_1d_8192", 2, 3, 2, (8192,), (16,)),                 # a long 1-D signal: 64 chunks of 64 pairs
    ("l_1d_1040_ragged", 1, 3, 1, (1040,), (32,)),          # 65 k-steps: a last chunk of one k-step; 3 rows; 32 modes
    ("l_2d_1024", 1, 1, 2, (24, 1024), (8, 12)),            # 24 rows per channel, k3 = 12 (frequencies past k3 idle)
    ("l_3d_528", 1, 2, 1, (6, 10, 528), (2, 4, 20)),        # three 8-frequency k-steps in the expansion
    ("l_1d_16384_k3", 1, 2, 2, (16384,), (3,)),              # the longest row, a few frequencies of one tile
    ("l_2d_600", 1, 2, 2, (16, 600), (4, 16)),              # 300 pairs: a last chunk of 44 (its last k-step half full)
    ("l_1d_1000", 2, 2, 1, (1000,), (20,)),                 # 500 pairs: a last chunk of 52
]


@pytest.mark.parametrize("case", LONG_ROWS, ids=[c[0] for c in LONG_ROWS])
def test_long_rows_run_on_the_chunked_row_kernels(case):
    name, B, Ci, Co, N, k = case
    w = I.custom_workload(name, B, Ci, Co, N, k, field="grf", seed=43)
    plan = _plan(w)
    assert plan.kernel_path == "row"
    plan.require_fast_path()
    plan.close()
    run_layer_and_check(w, "auto")
    run_layer_and_check(w, "auto", tol=2e-3, fine_scale=200.0, arithmetic="tf32")


@pytest.mark.parametrize("case", ANY_EXTENT, ids=[c[0] for c in ANY_EXTENT])
def test_any_contiguous_extent_runs_on_the_row_kernels(case):
    name, B, Ci, Co, N, k, streaming = case
    w = I.custom_workload(name, B, Ci, Co, N, k, field="grf", seed=31)
    plan = _plan(w)
    assert plan.kernel_path == "row"
    if streaming:
        plan.require_fast_path()
    plan.close()
    run_layer_and_check(w, "auto")
    if N[0] % 4 == 0 and len(N) > 1:
        run_layer_and_check(w, "auto", P=4)


# ------------------------------------------------------------------ single-pass TF32 arithmetic (a plan option)
@pytest.mark.parametrize("N,k", [((16, 16, 32, 30), (4, 8, 8, 16)),      # the paper's layer in small: fused plane kernels
                                 ((32, 45, 100), (6, 10, 12)),           # row kernel + middle kernels of any extent
                                 ((40, 90), (20, 17))])
def test_single_pass_tf32_meets_its_stated_error(N, k):
    """DTST_ARITH_TF32: every output within 2e-3 of the float64 statement (and not by accident on the compensated path:
    the error is well above that path's), the default arithmetic untouched."""
    w = I.custom_workload("tf32", 1, 2, 2, N, k, field="grf", seed=41)
    errs_fast = run_layer_and_check(w, "auto", tol=2e-3, fine_scale=200.0, arithmetic="tf32")
    errs = run_layer_and_check(w, "auto")
    for name in ("Xhat", "y", "grad_x", "grad_W"):
        assert errs_fast[name] > 10.0 * errs[name], (name, errs_fast, errs)


def test_arithmetic_option_rejects_unknown_modes():
    from paper_2607_14394_b200 import binding as Bn
    plan = _plan(I.WORKLOADS["cfg1_2d_64"])
    with pytest.raises(Bn.DtstError) as e:
        Bn.dtst_plan_set_arithmetic(plan.handle, 7)
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG
    plan.set_arithmetic("tf32")
    plan.set_arithmetic("tf32x3")
    plan.close()


# ------------------------------------------------------------------ third dimension inside the forward plane kernel
@pytest.mark.parametrize("N,k,B,C,P", [
    ((32, 128, 64), (16, 16, 8), 1, 3, 1),        # d = 3: the kernel writes the spectrum itself; N1 = 2 k1 (all of dim 0)
    ((64, 128, 64), (16, 16, 8), 2, 2, 1),        # four columns on four CTAs
    ((3, 128, 128, 64), (1, 16, 16, 8), 1, 1, 1), # N1 = 128: sixteen batches per column; a stage behind the kernel
    ((4, 64, 128, 64), (2, 16, 16, 8), 1, 2, 2),  # virtual shards on dimension 0 behind the fused kernel
])
def test_forward_with_the_third_dimension_fused(N, k, B, C, P):
    """Shapes whose forward-type transforms contract three dimensions in one kernel (columns of planes accumulated
    in the MMA fragments of extra warps): forward, inverse and backward against the oracle."""
    w = I.custom_workload("colfuse", B, C, C, N, k, field="grf", seed=47)
    plan = _plan(w, "auto", P, column_contraction=1)   # these cases have too few columns for the automatic choice
    assert plan.kernel_path == "fused"
    # one launch per forward: plane kernel (+ one per remaining dimension)
    before = plan.launch_count()
    plan.forward(_dev(I.make_field(w)))
    torch.cuda.synchronize()
    assert plan.launch_count() - before <= 1 + (len(N) - 3) + (1 if P > 1 else 0)   # (+ the slab reduction)
    # the automatic choice keeps the separate launch for so few columns (a CTA takes whole columns)
    auto = _plan(w, "auto", P)
    before = auto.launch_count()
    auto.forward(_dev(I.make_field(w)))
    torch.cuda.synchronize()
    assert auto.launch_count() - before >= 2 + (len(N) - 3)
    auto.close()
    plan.close()
    run_layer_and_check(w, "auto", P=P, column_contraction=1)


def test_fused_third_dimension_many_columns_is_reproducible():
    """More columns than SMs (some CTAs walk two columns, their batch buffers and accumulators are reused), three
    channels, N1 = 32: two runs give the same bits (the accumulation order is fixed), a run with the separate
    launch agrees within rounding, and the result meets the oracle."""
    w = I.custom_workload("colfuse_many", 1, 3, 3, (50, 32, 128, 64), (4, 16, 16, 8), field="grf", seed=53)
    x = _dev(I.make_field(w))
    fused = _plan(w, column_contraction=1)
    a = fused.forward(x).clone()
    b = fused.forward(x).clone()
    torch.cuda.synchronize()
    assert fused.status() == 0
    assert torch.equal(torch.view_as_real(a), torch.view_as_real(b))
    plain = _plan(w, column_contraction=-1)
    c = plain.forward(x)
    torch.cuda.synchronize()
    assert plain.launch_count() > 0 and O.rel_l2(a.cpu().numpy(), c.cpu().numpy()) <= 2e-6
    ref = O.forward(I.make_field(w), w.kmax)
    assert O.rel_l2(a.cpu().numpy(), ref) <= TOL
    assert per_mode_excess(a.cpu().numpy(), ref) <= 1.0
    fused.close()
    plain.close()


# ------------------------------------------------------------------ contraction order and pencils
@pytest.mark.parametrize("N,k,order", [
    ((32, 64, 16), (4, 8, 3), (0, 1)),                 # generic/folded: dimension 0 before dimension 1
    ((32, 64, 64, 32), (8, 4, 8, 4), (0, 2, 1)),       # fused: the plane kernel keeps dims 2, 3; 0 before 1
    ((16, 12, 8, 20), (2, 5, 3, 6), (1, 0, 2)),        # generic kernels, mixed
    ((6, 8), (3, 4), (0,)),
])
def test_any_contraction_order_gives_the_same_layer(N, k, order):
    """The result does not depend on the contraction order (Section "cuBLAS vs cuFFT"): every order meets the
    tolerance against the oracle, forward, inverse and backward."""
    w = I.custom_workload("order", 1, 2, 2, N, k, field="grf", seed=37)
    x, W, g = I.make_field(w), I.make_weights(w), I.make_upstream_grad(w)
    plan = _plan(w)
    default = plan.contraction_order()
    assert default == list(range(len(N) - 2, -1, -1))
    plan.set_contraction_order(order)
    assert plan.contraction_order() == list(order)
    Xhat = plan.forward(_dev(x))
    y = plan.inverse(plan.spectral_mul(Xhat, _dev(W)))
    gx, gW = plan.backward(_dev(g), Xhat, _dev(W))
    torch.cuda.synchronize()
    assert plan.status() == 0
    Wm = W.reshape((w.C_in, w.C_out) + w.K)
    y_ref, X_ref = O.layer_forward(x, Wm, w.kmax)
    gx_ref, gW_ref = O.backward(g, X_ref, Wm, w.kmax)
    assert O.rel_l2(Xhat.cpu().numpy(), X_ref) <= TOL and O.rel_l2(y.cpu().numpy(), y_ref) <= TOL
    assert O.rel_l2(gx.cpu().numpy(), gx_ref) <= TOL
    assert O.rel_l2(gW.cpu().numpy().reshape(gW_ref.shape), gW_ref) <= TOL


def test_order_tuner_contracts_the_most_compressing_dimension_first():
    from paper_2607_14394_b200 import Plan, binding as Bn
    # dimension 0 keeps 2*2 of 64 entries (ratio 1/16), dimension 1 keeps 2*12 of 32 (3/4): 0 should go first
    w = I.custom_workload("tune", 1, 2, 2, (64, 32, 16), (2, 12, 3), field="grf", seed=41)
    plan = _plan(w)
    before, after = plan.tune_contraction_order()
    assert plan.contraction_order() == [0, 1] and after < before
    # modelled bytes: 8 bytes per complex element read and written by every stage behind the grid-side kernel
    row = plan.kernel_path != "generic"
    k_last = w.K[-1]
    elems = lambda n0, n1: 2 * n0 * n1 * k_last
    want_after = 8 * (elems(64, 32) + elems(4, 32) + elems(4, 32) + elems(4, 24))
    want_before = 8 * (elems(64, 32) + elems(64, 24) + elems(64, 24) + elems(4, 24))
    assert (before, after) == (want_before, want_after), (row, before, after)
    run = plan.forward(_dev(I.make_field(w)))
    assert O.rel_l2(run.cpu().numpy(), O.forward(I.make_field(w), w.kmax)) <= TOL
    # with virtual shards dimension 0 has to stay last
    p2 = Plan(w.N, w.kmax, 1, 2, 2, virtual_shards=4)
    p2.tune_contraction_order()
    assert p2.contraction_order()[-1] == 0
    with pytest.raises(Bn.DtstError) as e:
        p2.set_contraction_order((0, 1))
    assert e.value.status == Bn.DTST_ERR_INVALID_ARG
    with pytest.raises(Bn.DtstError):
        plan.set_contraction_order((0, 0))


def test_pencil_block_runs_on_the_tensor_core_slab_kernels():
    """A rank's pencil (offsets on dimensions 0 AND 1, Section "Computing the Local Partial Spectrum") stays on the
    streaming family: plane kernel on the last two dimensions, slab kernels with global phases on the cut ones."""
    from paper_2607_14394_b200 import Plan
    Ng, k, nl, off = (64, 64, 64, 32), (8, 8, 8, 4), (16, 32, 64, 32), (32, 32, 0, 0)
    w = I.custom_workload("pencil", 1, 2, 2, Ng, k, field="grf", seed=43)
    x = I.make_field(w)
    blk = np.ascontiguousarray(x[:, :, 32:48, 32:64])
    plan = Plan(nl, k, 1, 2, 2, N_global=Ng, offset=off)
    assert plan.kernel_path == "fused"
    plan.require_fast_path()
    part = plan.forward(_dev(blk)).cpu().numpy()
    assert O.rel_l2(part, O.forward(blk, k, N_global=Ng, offsets=off)) <= TOL
    Y = I.make_spectrum(w, 2, tag=5).reshape((1, 2) + part.shape[2:])
    yb = plan.inverse(_dev(Y)).cpu().numpy()
    assert O.rel_l2(yb, O.inverse(Y, Ng, k, n_local=nl, offsets=off)) <= TOL


def test_fast_path_or_fail():
    from paper_2607_14394_b200 import binding as Bn
    # 40 modes per side in the middle (the folded kernels stop at 32): the generic kernel would serve that dimension
    w = I.custom_workload("slowmid", 1, 2, 2, (96, 64, 64), (40, 8, 8))
    plan = _plan(w)
    with pytest.raises(Bn.DtstError) as e:
        plan.require_fast_path()
    assert e.value.status == Bn.DTST_ERR_UNSUPPORTED
    plan.forward(_dev(I.make_field(w)))                      # not required: still runs (on the generic kernel)
    # all stages streaming: accepted; switching the plan to the generic family afterwards makes the calls refuse
    w2 = I.WORKLOADS["cfg3_4d_64"]
    p2 = _plan(w2)
    p2.require_fast_path()
    x2 = _dev(I.make_field(w2))
    p2.forward(x2)
    Bn.dtst_plan_set_kernel_path(p2.handle, Bn.DTST_PATH_GENERIC)
    before = p2.launch_count()
    with pytest.raises(Bn.DtstError) as e:
        p2.forward(x2)
    assert e.value.status == Bn.DTST_ERR_UNSUPPORTED and p2.launch_count() == before
    p2.require_fast_path(False)
    p2.forward(x2)
    # the row family counts as fast as well
    p4 = _plan(I.WORKLOADS["cfg2_3d_64"])
    assert p4.kernel_path == "row"
    p4.require_fast_path()


def test_adjoint_identity_on_device():
    # <F x, Y> = <x, F^H Y> holds for the kernels themselves at a size the oracle need not touch
    w = I.custom_workload("adj", 1, 2, 2, (32, 32, 64), (4, 6, 8), seed=77)
    plan = _plan(w)
    x = torch.randn((1, 2) + w.N, device="cuda", generator=torch.Generator("cuda").manual_seed(1))
    Y = torch.randn((1, 2) + w.K, dtype=torch.complex64, device="cuda",
                    generator=torch.Generator("cuda").manual_seed(2))
    Fx = plan.forward(x)
    lhs = (Fx.conj() * Y).real.double().sum().item()
    # F^H is not exposed on its own; I(Y) = F^H(c * Y) / prod(N), so divide the doubling weights out first
    c = torch.full((w.K[-1],), 2.0, device="cuda")
    c[0] = 1.0
    Yc = (Y / c).contiguous()
    rhs = (x.double() * plan.inverse(Yc).double()).sum().item() * float(np.prod(w.N))
    assert abs(lhs - rhs) <= 1e-5 * max(1.0, abs(lhs))


def test_step_can_be_captured_in_a_cuda_graph():
    # the compute calls allocate nothing and never synchronise: a whole step captures as it is and replays bit for bit
    w = I.custom_workload("graph", 2, 3, 2, (32, 32, 64), (4, 8, 8), field="grf", seed=41)
    plan = _plan(w)
    x, W, g = _dev(I.make_field(w)), _dev(I.make_weights(w)), _dev(I.make_upstream_grad(w))
    X = plan.forward(x)
    Y = plan.spectral_mul(X, W)
    y = plan.inverse(Y)
    gx, gW = plan.backward(g, X, W)

    def step():
        plan.forward(x, X)
        plan.spectral_mul(X, W, Y)
        plan.inverse(Y, y)
        plan.backward(g, X, W, gx, gW)

    step()
    torch.cuda.synchronize()
    ref = [t.clone() for t in (X, Y, y, gx, gW)]
    side, graph = torch.cuda.Stream(), torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        step()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph, stream=side):
            step()
    torch.cuda.synchronize()
    for t in (X, Y, y, gx, gW):
        t.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert plan.status() == 0
    for got, want in zip((X, Y, y, gx, gW), ref):
        assert torch.equal(torch.view_as_real(got) if got.is_complex() else got,
                           torch.view_as_real(want) if want.is_complex() else want)


def test_host_pipeline_matches_device_path_over_consecutive_steps():
    # pinned host buffers in and out, copies overlapped with compute on three streams: same bits as the plain path
    from paper_2607_14394_b200 import Plan
    from paper_2607_14394_b200.binding import HostPipeline
    w = I.custom_workload("hostpipe", 1, 2, 2, (16, 16, 64, 32), (2, 3, 8, 4), field="grf", seed=61)
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
    Wd = _dev(I.make_weights(w))
    pipe = HostPipeline(plan, Wd)
    outs = []
    for rep in range(3):
        wv = I.custom_workload("hostpipe", 1, 2, 2, w.N, w.kmax, field="grf", seed=61 + rep)
        hx = torch.from_numpy(I.make_field(wv)).pin_memory()
        hg = torch.from_numpy(I.make_upstream_grad(wv)).pin_memory()
        hy, hgx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
        hgW = torch.empty((w.C_in, w.C_out, w.M), dtype=torch.complex64).pin_memory()
        pipe.step(hx, hg, hy, hgx, hgW)
        outs.append((hx, hg, hy, hgx, hgW))
    pipe.wait()
    torch.cuda.synchronize()
    ref_plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
    for hx, hg, hy, hgx, hgW in outs:
        y, Xhat = ref_plan.layer(hx.cuda(), Wd)
        gx, gW = ref_plan.backward(hg.cuda(), Xhat, Wd)
        torch.cuda.synchronize()
        assert torch.equal(hy, y.cpu()) and torch.equal(hgx, gx.cpu())
        assert torch.equal(torch.view_as_real(hgW), torch.view_as_real(gW.cpu()))
    # and the first of them against the oracle
    hx, hg, hy, hgx, hgW = outs[0]
    y_ref, X_ref = O.layer_forward(hx.numpy(), Wd.cpu().numpy(), w.kmax)
    assert O.rel_l2(hy.numpy(), y_ref) <= TOL
