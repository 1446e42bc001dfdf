"""The truncated spectral layer across the ranks of one process group, the way Algorithm 1 shards it:

* the grid is cut into slabs along dimension 0; rank p owns slab p and transforms it with the global phase
  offsets of Eq. 18, which gives the PARTIAL spectrum of Eq. 6;
* an all-reduce (sum) of the partial spectra gives every rank the full spectrum (Eq. 7);
* rank p mixes its equal, contiguous share S_p of the flattened modes with its shard of the weights (Eq. 12);
* an all-gather of the mixed chunks gives every rank the full mixed spectrum, which it expands on its own slab
  (Eq. 14) - no further exchange;
* backward mirrors this: partial gradient spectrum, all-reduce, adjoint mixing on the rank's modes (the weight
  gradient of a shard is complete on its rank: no all-reduce of weight gradients), all-gather, local expansion.

Two collectives per direction, each of one spectrum (B * C * M complex values: 33.6 MB at the benchmark's largest
configuration).  The collectives are torch.distributed's (NCCL on GPUs); all compute runs in the CUDA library through
`Plan`.  The compute steps are also exposed one by one (`local_*`) so that the exchange can be driven by hand.

`ops` exists for tests only: the collective logic can be exercised on CPU ranks (gloo) with a stand-in for the
CUDA steps.  The default (`ops=None`) is the CUDA library and fails loudly without it.
"""
from __future__ import annotations

import math
from typing import Optional, Sequence, Tuple

import torch


def mode_counts(N: Sequence[int], kmax: Sequence[int]) -> Tuple[Tuple[int, ...], int]:
    """Retained modes per dimension (two-sided 2k on all but the last, k on the last) and their product."""
    d = len(N)
    K = tuple(2 * int(kmax[j]) if j < d - 1 else int(kmax[j]) for j in range(d))
    return K, math.prod(K)


class _CudaOps:
    """The six local steps on the CUDA library for one rank's slab."""

    def __init__(self, N_global, n_local, offset, kmax, B, C_in, C_out, device):
        from .binding import Plan
        self.plan = Plan(n_local, kmax, B, C_in, C_out, N_global=N_global, offset=offset, device=device)
        self.B, self.C_in, self.C_out, self.M = B, C_in, C_out, self.plan.M
        self.K = self.plan.K

    def spectrum(self, x_local):
        return self.plan.forward(x_local).reshape(self.B, self.C_in, self.M)

    def mix(self, Xhat, W_shard, m0, cnt):
        return self.plan.spectral_mul_modes(Xhat, W_shard, m0, cnt)

    def inverse(self, Yhat):
        return self.plan.inverse(Yhat.reshape((self.B, self.C_out) + self.K))

    def grad_spectrum(self, g_local):
        return self.plan.backward_spectrum(g_local).reshape(self.B, self.C_out, self.M)

    def grad_mix(self, GY, Xhat, W_shard, m0, cnt):
        return self.plan.backward_mix_modes(GY, Xhat, W_shard, m0, cnt)

    def grad_input(self, GX):
        return self.plan.backward_input(GX.reshape((self.B, self.C_in) + self.K))


class SlabShardedLayer:
    """One rank's view of the slab-sharded layer.  `world` must divide N_global[0] and the mode count M."""

    def __init__(self, N_global: Sequence[int], kmax: Sequence[int], B: int, C_in: int, C_out: int, world: int,
                 rank: int, device=None, ops=None):
        N_global = tuple(int(n) for n in N_global)
        if world < 1 or not (0 <= rank < world):
            raise ValueError("bad world / rank")
        if N_global[0] % world != 0:
            raise ValueError("the number of ranks must divide the extent of dimension 0 (equal slabs)")
        self.K, self.M = mode_counts(N_global, kmax)
        if self.M % world != 0:
            raise ValueError("the number of ranks must divide the number of retained modes (equal partition S_p)")
        self.world, self.rank = world, rank
        self.B, self.C_in, self.C_out = B, C_in, C_out
        self.N_global = N_global
        self.n_local = (N_global[0] // world,) + N_global[1:]
        self.offset = (rank * self.n_local[0],) + (0,) * (len(N_global) - 1)
        self.cnt = self.M // world
        self.m0 = rank * self.cnt
        self.ops = ops if ops is not None else _CudaOps(N_global, self.n_local, self.offset, tuple(kmax), B, C_in,
                                                        C_out, device)

    # ---- local steps -------------------------------------------------------------------------------------
    def local_spectrum(self, x_local):
        """Partial spectrum of this rank's slab, [B, C_in, M] (Eq. 6 with the offset basis of Eq. 18)."""
        return self.ops.spectrum(x_local)

    def local_mix(self, Xhat_full, W_shard):
        """This rank's chunk of the mixed spectrum, [B, C_out, M / world] (Eq. 12 on S_p)."""
        return self.ops.mix(Xhat_full, W_shard, self.m0, self.cnt)

    def local_inverse(self, Yhat_full):
        """y on this rank's slab from the full mixed spectrum (Eq. 14)."""
        return self.ops.inverse(Yhat_full)

    def local_grad_spectrum(self, g_local):
        return self.ops.grad_spectrum(g_local)

    def local_grad_mix(self, GY_full, Xhat_full, W_shard):
        """(G_X chunk [B, C_in, M / world], grad_W shard [C_in, C_out, M / world])."""
        return self.ops.grad_mix(GY_full, Xhat_full, W_shard, self.m0, self.cnt)

    def local_grad_input(self, GX_full):
        return self.ops.grad_input(GX_full)

    # ---- chunk assembly ----------------------------------------------------------------------------------
    @staticmethod
    def assemble(chunks: torch.Tensor) -> torch.Tensor:
        """[world, B, C, cnt] (rank-major, as an all-gather delivers it) -> [B, C, world * cnt]."""
        P, B, C, cnt = chunks.shape
        return chunks.permute(1, 2, 0, 3).reshape(B, C, P * cnt).contiguous()

    # ---- collectives -------------------------------------------------------------------------------------
    def _all_reduce(self, t: torch.Tensor, group) -> torch.Tensor:
        import torch.distributed as dist
        if self.world > 1:
            dist.all_reduce(torch.view_as_real(t), op=dist.ReduceOp.SUM, group=group)
        return t

    def _all_gather(self, chunk: torch.Tensor, group) -> torch.Tensor:
        import torch.distributed as dist
        chunk = chunk.contiguous()
        # rank-major concatenation along dimension 0 (the layout every backend accepts), viewed as [world, ...]
        out = torch.empty((self.world * chunk.shape[0],) + tuple(chunk.shape[1:]), dtype=chunk.dtype,
                          device=chunk.device)
        if self.world > 1:
            dist.all_gather_into_tensor(torch.view_as_real(out), torch.view_as_real(chunk), group=group)
        else:
            out.copy_(chunk)
        return self.assemble(out.view((self.world,) + tuple(chunk.shape)))

    def forward(self, x_local, W_shard, group=None):
        """Returns (y on this rank's slab, the full spectrum Xhat to keep for backward)."""
        Xhat = self._all_reduce(self.local_spectrum(x_local), group)
        Yhat = self._all_gather(self.local_mix(Xhat, W_shard), group)
        return self.local_inverse(Yhat), Xhat

    def backward(self, g_local, Xhat_full, W_shard, group=None):
        """Returns (grad_x on this rank's slab, grad_W for this rank's modes)."""
        GY = self._all_reduce(self.local_grad_spectrum(g_local), group)
        GX_chunk, gW_shard = self.local_grad_mix(GY, Xhat_full, W_shard)
        GX = self._all_gather(GX_chunk, group)
        return self.local_grad_input(GX), gW_shard


def shard_weights(W: torch.Tensor, world: int, rank: int) -> torch.Tensor:
    """Rank `rank`'s contiguous share of the modes of W [C_in, C_out, M] -> [C_in, C_out, M / world]."""
    M = W.shape[-1]
    if M % world != 0:
        raise ValueError("the number of ranks must divide the number of retained modes")
    cnt = M // world
    return W[..., rank * cnt:(rank + 1) * cnt].contiguous()
