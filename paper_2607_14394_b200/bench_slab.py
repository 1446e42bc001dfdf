"""Timing of the slab-sharded layer (Algorithm 1) over the GPUs of one node: one process per GPU,
`python -m torch.distributed.run --nnodes=1 --nproc-per-node N --master-addr 127.0.0.1 -m
paper_2607_14394_b200.bench_slab --config cfg5_4d_128`, or plain `python -m paper_2607_14394_b200.bench_slab` for
one GPU (then the collectives are skipped and the step is the step-wise path of one rank).

STRONG scaling: the global grid of the configuration is cut into N slabs along dimension 0, the modes and the
weights into N equal chunks; per step every rank runs forward + backward of the layer with two NCCL collectives
per direction (all-reduce of the partial spectrum, all-gather of the mixed chunks).  Timed with CUDA events after
warm-up, between barriers, max over ranks; rank 0 prints one JSON line.  This is a companion to bench.py (whose
multi-GPU mode shards independent batches and needs no collective), not part of its contract.
"""
from __future__ import annotations

import argparse
import json

import torch


def main() -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="cfg5_4d_128")
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()

    from . import dist as D
    from . import inputs
    from .dist_layer import SlabShardedLayer

    if not torch.cuda.is_available():
        raise RuntimeError("bench_slab needs CUDA devices (the layer has no CPU path)")
    world, rank, local_rank = D.env_world()
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    D.init_process_group("nccl", dev)
    w = inputs.WORKLOADS[args.config]
    layer = SlabShardedLayer(w.N, w.kmax, w.B, w.C_in, w.C_out, world, rank, device=dev)

    gen = torch.Generator(device=dev)
    gen.manual_seed(D.rank_seed(w.seed, rank))
    x = torch.randn((w.B, w.C_in) + layer.n_local, generator=gen, device=dev)
    g = torch.randn((w.B, w.C_out) + layer.n_local, generator=gen, device=dev)
    W_shard = torch.view_as_complex(torch.randn((w.C_in, w.C_out, layer.cnt, 2), generator=gen, device=dev)
                                    / (w.C_in * w.C_out) ** 0.5)

    def step():
        y, Xhat = layer.forward(x, W_shard)
        gx, gW = layer.backward(g, Xhat, W_shard)
        return y, gx, gW

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    if layer.ops.plan.status() != 0:
        raise RuntimeError("device-side status word set during warm-up")
    launches0 = layer.ops.plan.launch_count()
    barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    barrier()
    ms = D.max_over_ranks([e0.elapsed_time(e1) / args.steps], device=dev)[0]
    launches = layer.ops.plan.launch_count() - launches0
    if rank == 0:
        pts = w.B * w.points                       # the GLOBAL grid: total work is fixed as N grows
        print(json.dumps({
            "metric": "spectral_layer_fwd_bwd_grid_points_per_s", "value": pts / (ms * 1e-3) / 1e9,
            "unit": "Gpoints/s", "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "grid": list(w.N), "kmax": list(w.kmax), "slab": list(layer.n_local),
                       "modes_per_rank": layer.cnt,
                       "parallelism": f"slab{world}: all-reduce + all-gather of one spectrum per direction (NCCL)"},
            "gpu_launches": int(launches),
            "collective_bytes_per_step": 0 if world == 1 else
            8 * w.B * w.M * (2 * w.C_in + 2 * w.C_out)}))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
