"""A whole Fourier neural operator on one GPU, sequenced from the library's C-ABI calls.

Section "Background and Motivation" of the paper: the input a is lifted to d_v channels by a point-wise network
P, passed through L Fourier layers v -> GELU(W_bypass v + I(M(F(v), W))) (Eq. 1; Algorithm 1 without the
collectives) and projected back by a point-wise network Q.  P and Q are one linear map with bias each.  This
module only orders the calls and owns the buffers: every arithmetic step runs in the CUDA library
(dtst_pointwise_linear, dtst_block_forward, dtst_block_backward, dtst_pointwise_linear_backward).  There is no
PyTorch or CPU fallback.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch

from . import binding as Bn


class FNO:
    """forward(a) -> u and backward(grad_u) -> gradients of every parameter, for a fixed batch and grid.

    a [B, C_a, n...] float32, u [B, C_u, n...]; `width` = d_v channels inside; `layers` Fourier layers.
    Parameters are plain tensors owned by this object: P_w [d_v, C_a], P_b [d_v], per layer W [d_v, d_v, M]
    complex64 and W_bypass [d_v, d_v], Q_w [C_u, d_v], Q_b [C_u].
    """

    def __init__(self, N: Sequence[int], kmax: Sequence[int], B: int, C_a: int, C_u: int, width: int, layers: int,
                 device=None, seed: int = 0, arithmetic: str = "tf32x3"):
        self.plan = Bn.Plan(N, kmax, B, width, width, device=device, arithmetic=arithmetic)
        dev = self.plan.device
        self.N, self.B, self.C_a, self.C_u, self.width, self.layers = tuple(N), B, C_a, C_u, width, layers
        gen = torch.Generator(device=dev).manual_seed(seed)
        rn = lambda *shape: torch.randn(shape, device=dev, generator=gen)
        M = self.plan.M
        self.P_w, self.P_b = rn(width, C_a) / C_a ** 0.5, rn(width) * 0.1
        self.Q_w, self.Q_b = rn(C_u, width) / width ** 0.5, rn(C_u) * 0.1
        self.W: List[torch.Tensor] = [torch.view_as_complex(rn(width, width, M, 2) / width).contiguous()
                                      for _ in range(layers)]
        self.Wb: List[torch.Tensor] = [rn(width, width) / width ** 0.5 for _ in range(layers)]
        grid = (B, width) + self.N
        # activations kept for the backward pass: the input of every layer, its pre-activation and its spectrum
        self.v = [torch.empty(grid, device=dev) for _ in range(layers + 1)]
        self.z = [torch.empty(grid, device=dev) for _ in range(layers)]
        self.Xhat = [torch.empty((B, width) + self.plan.K, dtype=torch.complex64, device=dev) for _ in range(layers)]
        self.u = torch.empty((B, C_u) + self.N, device=dev)
        self.g = [torch.empty(grid, device=dev) for _ in range(2)]      # gradient ping-pong
        nscratch = max(Bn.dtst_pointwise_linear_scratch_bytes(C_a, width),
                       Bn.dtst_pointwise_linear_scratch_bytes(width, C_u))
        self.scratch = torch.empty(nscratch, dtype=torch.uint8, device=dev)
        self.a = None

    def forward(self, a: torch.Tensor, stream=None) -> torch.Tensor:
        self.a = a
        Bn.dtst_pointwise_linear(a, self.P_w, self.P_b, self.v[0], stream)
        for l in range(self.layers):
            self.plan.block_forward(self.v[l], self.W[l], self.Wb[l], self.v[l + 1], self.Xhat[l], self.z[l],
                                    stream=stream)
        Bn.dtst_pointwise_linear(self.v[self.layers], self.Q_w, self.Q_b, self.u, stream)
        return self.u

    def backward(self, grad_u: torch.Tensor, need_grad_a: bool = False, stream=None) -> dict:
        dev = self.plan.device
        grads = {"Q_w": torch.empty_like(self.Q_w), "Q_b": torch.empty_like(self.Q_b),
                 "P_w": torch.empty_like(self.P_w), "P_b": torch.empty_like(self.P_b), "W": [], "Wb": []}
        g, other = self.g
        Bn.dtst_pointwise_linear_backward(grad_u, self.v[self.layers], self.Q_w, g, grads["Q_w"], grads["Q_b"],
                                          self.scratch, stream)
        for l in reversed(range(self.layers)):
            gW = torch.empty_like(self.W[l])
            gWb = torch.empty_like(self.Wb[l])
            # g is overwritten with g_z (it is this layer's scratch) and the input gradient lands in `other`
            self.plan.block_backward(g, self.v[l], self.z[l], self.Xhat[l], self.W[l], self.Wb[l], scratch=g,
                                     grad_x=other, grad_W=gW, grad_W_bypass=gWb, stream=stream)
            grads["W"].insert(0, gW)
            grads["Wb"].insert(0, gWb)
            g, other = other, g
        ga = torch.empty_like(self.a) if need_grad_a else None
        Bn.dtst_pointwise_linear_backward(g, self.a, self.P_w, ga, grads["P_w"], grads["P_b"], self.scratch, stream)
        grads["a"] = ga
        return grads

    def parameters(self) -> Tuple:
        return (self.P_w, self.P_b, self.W, self.Wb, self.Q_w, self.Q_b)

    def close(self):
        self.plan.close()
