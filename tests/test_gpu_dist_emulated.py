"""The slab-sharded layer's CUDA steps on ONE GPU: P virtual ranks run one after the other (no kernel waits on
another), the all-reduce is a sum in ascending rank order and the all-gather a concatenation, both done by hand.
What is checked is the part the gloo test cannot reach: the local plans with global offsets, the chunked mixing
kernels with sharded weights, and the step-wise backward entry points, all through the C ABI against the oracle."""
import numpy as np
import pytest

from oracle import dtst_oracle as O
from paper_2607_14394_b200 import inputs as I

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


@pytest.mark.parametrize("N,k,P", [((16, 8, 12), (3, 2, 4), 2), ((64, 32, 64), (8, 4, 8), 4),
                                   ((32, 32, 32, 32), (4, 4, 4, 4), 8), ((64, 64), (8, 8), 2)])
def test_virtual_ranks_match_oracle(N, k, P):
    from paper_2607_14394_b200.dist_layer import SlabShardedLayer, shard_weights
    dev = torch.device("cuda")
    w = I.custom_workload("dist_emulated", 2, 3, 2, N, k, field="grf", seed=101)
    x, W, g = I.make_field(w), I.make_weights(w), I.make_upstream_grad(w)
    Wd = torch.from_numpy(W).to(dev).reshape(w.C_in, w.C_out, w.M)
    layers = [SlabShardedLayer(N, k, w.B, w.C_in, w.C_out, P, r, device=dev) for r in range(P)]
    nl = N[0] // P
    slab = lambda a, r: torch.from_numpy(np.ascontiguousarray(a[:, :, r * nl:(r + 1) * nl])).to(dev)
    shards = [shard_weights(Wd, P, r) for r in range(P)]

    # forward: partial spectra -> "all-reduce" -> chunked mixing -> "all-gather" -> local expansion
    parts = [L.local_spectrum(slab(x, r)) for r, L in enumerate(layers)]
    Xhat = parts[0].clone()
    for p in parts[1:]:
        Xhat += p
    chunks = torch.stack([L.local_mix(Xhat, shards[r]) for r, L in enumerate(layers)])
    Yhat = SlabShardedLayer.assemble(chunks)
    y = torch.cat([L.local_inverse(Yhat) for L in layers], dim=2)
    y_ref, X_ref = O.layer_forward(x, W, w.kmax)
    assert O.rel_l2(Xhat.cpu().numpy(), X_ref.reshape(w.B, w.C_in, w.M)) <= TOL
    assert O.rel_l2(y.cpu().numpy(), y_ref) <= TOL

    # backward, mirrored; the weight gradient of a shard is complete on its rank
    gparts = [L.local_grad_spectrum(slab(g, r)) for r, L in enumerate(layers)]
    GY = gparts[0].clone()
    for p in gparts[1:]:
        GY += p
    mixed = [L.local_grad_mix(GY, Xhat, shards[r]) for r, L in enumerate(layers)]
    GX = SlabShardedLayer.assemble(torch.stack([m[0] for m in mixed]))
    gx = torch.cat([L.local_grad_input(GX) for L in layers], dim=2)
    gW = torch.cat([m[1] for m in mixed], dim=2)
    torch.cuda.synchronize()
    for L in layers:
        assert L.ops.plan.status() == 0
    gx_ref, gW_ref = O.backward(g, X_ref, W.reshape((w.C_in, w.C_out) + w.K), w.kmax)
    assert O.rel_l2(gx.cpu().numpy(), gx_ref) <= TOL
    assert O.rel_l2(gW.cpu().numpy(), gW_ref.reshape(w.C_in, w.C_out, w.M)) <= TOL


def test_step_entry_points_equal_the_fused_backward():
    """dtst_backward == dtst_backward_spectrum -> dtst_backward_mix_modes (all modes) -> dtst_backward_input."""
    from paper_2607_14394_b200 import Plan
    dev = torch.device("cuda")
    w = I.custom_workload("steps", 2, 2, 3, (32, 32, 64), (4, 4, 8), seed=5)
    x, W, g = (torch.from_numpy(a).to(dev) for a in (I.make_field(w), I.make_weights(w), I.make_upstream_grad(w)))
    plan = Plan(w.N, w.kmax, w.B, w.C_in, w.C_out)
    Xhat = plan.forward(x)
    gx_a, gW_a = plan.backward(g, Xhat, W)
    GY = plan.backward_spectrum(g)
    GXc, gW_b = plan.backward_mix_modes(GY.reshape(w.B, w.C_out, w.M), Xhat.reshape(w.B, w.C_in, w.M),
                                        W.reshape(w.C_in, w.C_out, w.M), 0, w.M)
    gx_b = plan.backward_input(GXc)
    Y_a = plan.spectral_mul(Xhat, W)
    Y_b = plan.spectral_mul_modes(Xhat.reshape(w.B, w.C_in, w.M), W.reshape(w.C_in, w.C_out, w.M), 0, w.M)
    torch.cuda.synchronize()
    rel = lambda a, b: float((a.double() - b.double()).norm() / b.double().norm()) if not a.is_complex() else \
        float((torch.view_as_real(a).double() - torch.view_as_real(b).double()).norm() /
              torch.view_as_real(b).double().norm())
    assert rel(gx_b, gx_a) <= 1e-6
    assert rel(gW_b.reshape(-1), gW_a.reshape(-1)) <= 1e-6
    assert rel(Y_b.reshape(-1), Y_a.reshape(-1)) <= 1e-6
    with pytest.raises(Exception):
        plan.spectral_mul_modes(Xhat.reshape(w.B, w.C_in, w.M), W.reshape(w.C_in, w.C_out, w.M), w.M - 1, 2)
