"""dtst_forward_static: the forward transform for callers that cannot allocate.

Some users of this library run where device allocation is off limits at call
time (a plug-in inside an application that owns all GPU memory, a loop that
bans allocator calls after start-up) and have no workspace to pass either.
For them the library keeps a fixed 8 MiB scratch array of its own.  This test
calls that entry point through the C ABI twice in a row and compares both
results with the ordinary dtst_forward and with the float64 oracle, with the
tolerance of the parity tests.
The file sorts last on purpose: if it fails, every other test has already run.
"""
import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import inputs as I

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


def _rel_l2(a, b):
    a = torch.view_as_real(a).double()
    b = torch.view_as_real(b).double()
    return float((a - b).norm() / b.norm())


@pytest.mark.parametrize("P", [1, 4])
def test_static_scratch_forward_matches_workspace_forward_twice(P):
    from paper_2607_14394_b200 import Plan
    w = I.custom_workload("noalloc", 2, 3, 2, (16, 24, 40), (3, 5, 6), field="grf", seed=41)
    x = torch.from_numpy(I.make_field(w)).cuda()
    ref_plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P)
    ref = ref_plan.forward(x)
    # the plan used with the static entry point never receives a workspace
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, virtual_shards=P, allocate_workspace=False)
    out1 = torch.full_like(ref, complex("nan+nanj"))
    out2 = torch.full_like(ref, complex("nan+nanj"))
    plan.forward_static(x, out1)
    # a different shape in between leaves other contents in the shared array
    w2 = I.custom_workload("noalloc2", 1, 2, 2, (8, 8, 64), (2, 3, 9), seed=42)
    x2 = torch.from_numpy(I.make_field(w2)).cuda()
    p2 = Plan(w2.N, w2.kmax, w2.B, w2.C_in, w2.C_out, allocate_workspace=False)
    o2 = torch.empty((w2.B, w2.C_in) + w2.K, dtype=torch.complex64, device="cuda")
    p2.forward_static(x2, o2)
    plan.forward_static(x, out2)
    torch.cuda.synchronize()
    assert _rel_l2(out1, ref) <= TOL
    assert _rel_l2(out2, ref) <= TOL
    # and against the oracle itself, not only against the sibling entry point
    X_ref = O.forward_sharded(I.make_field(w), w.kmax, P) if P > 1 else O.forward(I.make_field(w), w.kmax)
    assert O.rel_l2(out1.cpu().numpy(), X_ref) <= TOL
    assert O.rel_l2(out2.cpu().numpy(), X_ref) <= TOL
    ref2 = Plan(w2.N, w2.kmax, w2.B, w2.C_in, w2.C_out).forward(x2)
    assert _rel_l2(o2, ref2) <= TOL
    assert O.rel_l2(o2.cpu().numpy(), O.forward(I.make_field(w2), w2.kmax)) <= TOL


def test_static_scratch_limit_is_reported_not_exceeded():
    from paper_2607_14394_b200 import Plan, binding as Bn
    w = I.WORKLOADS["cfg2_3d_64"]     # first-stage intermediate alone is 12.6 MB > 8 MiB
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out, allocate_workspace=False)
    x = torch.zeros((w.B, w.C_in) + w.N, device="cuda")
    out = torch.zeros((w.B, w.C_in) + w.K, dtype=torch.complex64, device="cuda")
    before = plan.launch_count()
    with pytest.raises(Bn.DtstError) as e:
        plan.forward_static(x, out)
    assert e.value.status == Bn.DTST_ERR_STATIC_LIMIT
    assert "fixed scratch" in str(e.value)
    assert plan.launch_count() == before      # nothing was launched
