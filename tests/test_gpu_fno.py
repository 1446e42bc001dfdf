"""A whole synthetic FNO (lift, Fourier layers with bypass and GELU, projection) on the GPU, forward and
backward, every step in the library's kernels, against the float64 oracle with the same seeded parameters."""
import numpy as np
import pytest

from oracle import dtst_oracle as O

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

TOL = 1e-5


@pytest.mark.parametrize("N,kmax,B,Ca,Cu,width,layers", [
    ((16, 16, 32), (4, 4, 8), 2, 3, 2, 8, 2),
    ((32, 64, 64, 32), (4, 8, 8, 4), 1, 5, 1, 16, 3),     # plane + folded kernels, tensor-core-eligible width
    ((12, 20), (3, 5), 2, 1, 1, 5, 1),                     # odd width, generic kernels
])
def test_fno_forward_backward_match_the_oracle(N, kmax, B, Ca, Cu, width, layers):
    from paper_2607_14394_b200 import FNO
    net = FNO(N, kmax, B, Ca, Cu, width, layers, seed=123)
    gen = torch.Generator(device="cuda").manual_seed(7)
    a = torch.randn((B, Ca) + tuple(N), device="cuda", generator=gen)
    gu = torch.randn((B, Cu) + tuple(N), device="cuda", generator=gen)
    u = net.forward(a).clone()
    grads = net.backward(gu, need_grad_a=True)
    torch.cuda.synchronize()
    assert net.plan.status() == 0
    host = lambda t: t.detach().cpu().numpy()
    K = net.plan.K
    params = {"P_w": host(net.P_w), "P_b": host(net.P_b), "Q_w": host(net.Q_w), "Q_b": host(net.Q_b),
              "blocks": [(host(net.W[l]).reshape((width, width) + K), host(net.Wb[l])) for l in range(layers)]}
    u_ref, saved = O.fno_forward(host(a), params, kmax)
    g_ref = O.fno_backward(host(gu), params, saved, kmax)
    errs = {"u": O.rel_l2(host(u), u_ref), "a": O.rel_l2(host(grads["a"]), g_ref["a"])}
    for name in ("P_w", "P_b", "Q_w", "Q_b"):
        errs[name] = O.rel_l2(host(grads[name]), g_ref[name])
    for l in range(layers):
        errs[f"W{l}"] = O.rel_l2(host(grads["W"][l]).reshape(g_ref["blocks"][l][0].shape), g_ref["blocks"][l][0])
        errs[f"Wb{l}"] = O.rel_l2(host(grads["Wb"][l]), g_ref["blocks"][l][1])
    for name, e in errs.items():
        assert e <= TOL, (name, e, errs)
    # a second pass gives the same bits (every reduction runs in a fixed order)
    u2 = net.forward(a).clone()
    grads2 = net.backward(gu)
    torch.cuda.synchronize()
    assert torch.equal(u, u2) and torch.equal(grads["P_w"], grads2["P_w"]) and torch.equal(grads["Q_b"], grads2["Q_b"])
    net.close()


def test_pointwise_linear_argument_errors():
    from paper_2607_14394_b200 import binding as Bn
    x = torch.zeros((1, 3, 8, 8), device="cuda")
    W = torch.zeros((2, 3), device="cuda")
    out = torch.zeros((1, 2, 8, 8), device="cuda")
    Bn.dtst_pointwise_linear(x, W, None, out)
    with pytest.raises(ValueError):
        Bn.dtst_pointwise_linear(x, torch.zeros((2, 4), device="cuda"), None, out)
    with pytest.raises(Bn.DtstError) as e:       # weight gradient asked for without its scratch
        Bn.dtst_pointwise_linear_backward(out, x, W, None, torch.zeros_like(W), None, None)
    assert e.value.status == Bn.DTST_ERR_WORKSPACE


@pytest.mark.parametrize("B,Ci,Co,P", [
    (2, 16, 32, 1024),      # both products on the tensor cores: weight, bias and (assigned) input gradient
    (1, 32, 16, 128 * 37),  # an odd number of 128-point tiles, fewer tiles than CTAs
    (3, 32, 32, 4096),
    (2, 16, 16, 128 * 700), # more tiles than CTAs: every CTA walks several, partial sums over CTAs
    (2, 20, 20, 1024),      # the paper's width: channel counts padded to the MMA tiles inside the kernel
    (1, 8, 24, 128 * 5),
    (2, 12, 9, 256),
    (2, 5, 20, 1024),       # a lifting layer and a projection layer of the paper's FNO on the tensor cores
    (2, 20, 5, 1024),
    (1, 1, 32, 256),
    (1, 32, 1, 256),
    (2, 3, 16, 1000),       # points not a multiple of the tile, or few channels on both sides: the FFMA kernels
    (2, 16, 1, 520),        # ... and of a projection layer
])
def test_pointwise_linear_forward_and_backward(B, Ci, Co, P):
    """out = W x + b and the three gradients of a point-wise linear layer (Eq. 1: the lifting and projection
    networks; the block's bypass is the same operator without the bias) against float64 einsums."""
    from paper_2607_14394_b200 import binding as Bn
    rng = np.random.default_rng(1000 * Ci + Co)
    x = rng.standard_normal((B, Ci, P)).astype(np.float32)
    W = (rng.standard_normal((Co, Ci)) / np.sqrt(Ci)).astype(np.float32)
    b = rng.standard_normal(Co).astype(np.float32)
    g = rng.standard_normal((B, Co, P)).astype(np.float32)
    dev = lambda a: torch.from_numpy(a).cuda()
    xd, Wd, bd, gd = dev(x), dev(W), dev(b), dev(g)
    out = torch.empty((B, Co, P), device="cuda")
    Bn.dtst_pointwise_linear(xd, Wd, bd, out)
    ref = O.pointwise_linear(x, W, b)
    assert O.rel_l2(out.cpu().numpy(), ref) <= TOL
    scratch = torch.empty(Bn.dtst_pointwise_linear_scratch_bytes(Ci, Co), dtype=torch.uint8, device="cuda")
    gx = torch.full((B, Ci, P), float("nan"), device="cuda")
    gW = torch.full((Co, Ci), float("nan"), device="cuda")
    gb = torch.full((Co,), float("nan"), device="cuda")
    Bn.dtst_pointwise_linear_backward(gd, xd, Wd, gx, gW, gb, scratch)
    torch.cuda.synchronize()
    x64, g64, W64 = x.astype(np.float64), g.astype(np.float64), W.astype(np.float64)
    assert O.rel_l2(gx.cpu().numpy(), np.einsum("oi,bop->bip", W64, g64)) <= TOL
    assert O.rel_l2(gW.cpu().numpy(), np.einsum("bop,bip->oi", g64, x64)) <= TOL
    assert O.rel_l2(gb.cpu().numpy(), g64.sum(axis=(0, 2))) <= TOL
    # the same bits on a second run (fixed summation order), and the weight gradient alone
    gW2, gb2 = torch.empty_like(gW), torch.empty_like(gb)
    Bn.dtst_pointwise_linear_backward(gd, xd, Wd, None, gW2, gb2, scratch)
    torch.cuda.synchronize()
    assert torch.equal(gW, gW2) and torch.equal(gb, gb2)
