"""Stand-in for the CUDA library's six local steps of the slab-sharded layer, in float64 numpy on torch CPU
tensors.  Test infrastructure only: it lets world-size-2 gloo tests drive the real collectives and the real
exchange logic (offsets, chunk bounds, assembly order) on a machine without GPUs.  The product's steps are the
CUDA library's, covered by the GPU tests."""
import math

import numpy as np
import torch


class OracleOps:
    """The six local steps in float64 numpy, on torch CPU tensors."""

    def __init__(self, O, N_global, n_local, offset, kmax, B, C_in, C_out):
        if O is None:
            from oracle import dtst_oracle as O
        self.O, self.Ng, self.nl, self.off, self.k = O, tuple(N_global), tuple(n_local), tuple(offset), tuple(kmax)
        self.B, self.Ci, self.Co = B, C_in, C_out
        d = len(self.Ng)
        self.K = tuple(2 * self.k[j] if j < d - 1 else self.k[j] for j in range(d))
        self.M = math.prod(self.K)

    def spectrum(self, x):
        X = self.O.forward(x.numpy(), self.k, N_global=self.Ng, offsets=self.off)
        return torch.from_numpy(np.ascontiguousarray(X.reshape(self.B, self.Ci, self.M)))

    def mix(self, Xhat, W_shard, m0, cnt):
        Y = np.einsum("bim,iom->bom", Xhat.numpy()[:, :, m0:m0 + cnt], W_shard.numpy())
        return torch.from_numpy(np.ascontiguousarray(Y))

    def inverse(self, Yhat):
        y = self.O.inverse(Yhat.numpy().reshape((self.B, self.Co) + self.K), self.Ng, self.k, n_local=self.nl,
                           offsets=self.off)
        return torch.from_numpy(np.ascontiguousarray(y))

    def grad_spectrum(self, g):
        c = self.O.hermitian_weights(self.Ng[-1], self.k[-1])
        G = self.O.forward(g.numpy(), self.k, N_global=self.Ng, offsets=self.off) * c / float(math.prod(self.Ng))
        return torch.from_numpy(np.ascontiguousarray(G.reshape(self.B, self.Co, self.M)))

    def grad_mix(self, GY, Xhat, W_shard, m0, cnt):
        gy, xh = GY.numpy()[:, :, m0:m0 + cnt], Xhat.numpy()[:, :, m0:m0 + cnt]
        GX = np.einsum("bom,iom->bim", gy, np.conj(W_shard.numpy()))
        gW = np.einsum("bim,bom->iom", np.conj(xh), gy)
        return torch.from_numpy(np.ascontiguousarray(GX)), torch.from_numpy(np.ascontiguousarray(gW))

    def grad_input(self, GX):
        gx = self.O.inverse(GX.numpy().reshape((self.B, self.Ci) + self.K), self.Ng, self.k, n_local=self.nl,
                            offsets=self.off, doubling=False, normalise=False)
        return torch.from_numpy(np.ascontiguousarray(gx))


def make_ops(N_global, n_local, offset, kmax, B, C_in, C_out):
    """Factory with the signature bench.py's `--ops-module` option expects."""
    return OracleOps(None, N_global, n_local, offset, kmax, B, C_in, C_out)
