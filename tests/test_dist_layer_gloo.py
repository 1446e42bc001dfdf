"""World-size-2 gloo test (CPU) of the slab-sharded layer's exchange logic (Algorithm 1): partial spectra
all-reduced, modes partitioned in equal contiguous chunks with sharded weights, chunks all-gathered, and the same
mirrored for backward with no all-reduce of weight gradients.  The local compute steps are stood in for by the
float64 oracle (test infrastructure; the product's steps are the CUDA library's, covered by the GPU tests), so what
this test pins is the orchestration: offsets, chunk bounds, assembly order and the collectives."""
import math
import os
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


from gloo_ops import OracleOps


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import torch.distributed as dist
    from oracle import dtst_oracle as O
    from paper_2607_14394_b200 import dist as D
    from paper_2607_14394_b200.dist_layer import SlabShardedLayer, shard_weights
    assert D.init_process_group("gloo")
    try:
        N, k, B, Ci, Co = (8, 6, 10), (2, 3, 3), 2, 3, 2
        rng = np.random.default_rng(17)          # same seed on every rank: the global problem
        x = rng.standard_normal((B, Ci) + N)
        g = rng.standard_normal((B, Co) + N)
        K = (4, 6, 3)
        M = math.prod(K)
        W = (rng.standard_normal((Ci, Co, M)) + 1j * rng.standard_normal((Ci, Co, M))) / math.sqrt(Ci * Co)
        nl = N[0] // world
        ops = OracleOps(O, N, (nl,) + N[1:], (rank * nl, 0, 0), k, B, Ci, Co)
        layer = SlabShardedLayer(N, k, B, Ci, Co, world, rank, ops=ops)
        assert layer.offset == (rank * nl, 0, 0) and layer.cnt == M // world and layer.m0 == rank * (M // world)
        W_shard = shard_weights(torch.from_numpy(W), world, rank)
        sl = slice(rank * nl, (rank + 1) * nl)
        y_loc, Xhat = layer.forward(torch.from_numpy(np.ascontiguousarray(x[:, :, sl])), W_shard)
        gx_loc, gW_shard = layer.backward(torch.from_numpy(np.ascontiguousarray(g[:, :, sl])), Xhat, W_shard)
        # the single-process statement of the same layer on the whole grid
        y_ref, X_ref = O.layer_forward(x, W, k)
        gx_ref, gW_ref = O.backward(g, X_ref, W.reshape((Ci, Co) + K), k)
        assert O.rel_l2(Xhat.numpy(), X_ref.reshape(B, Ci, M)) < 1e-12
        assert O.rel_l2(y_loc.numpy(), y_ref[:, :, sl]) < 1e-12
        assert O.rel_l2(gx_loc.numpy(), gx_ref[:, :, sl]) < 1e-12
        cnt = M // world
        assert O.rel_l2(gW_shard.numpy(), gW_ref.reshape(Ci, Co, M)[:, :, rank * cnt:(rank + 1) * cnt]) < 1e-12
        q.put((rank, "ok"))
    except Exception as e:   # pragma: no cover
        import traceback
        q.put((rank, repr(e) + traceback.format_exc()))
    finally:
        dist.destroy_process_group()


def test_slab_sharded_layer_world_size_2_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=180) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
    assert sorted(results) == [(0, "ok"), (1, "ok")], results


def test_assemble_and_shard_bounds():
    sys.path.insert(0, ROOT)
    from paper_2607_14394_b200.dist_layer import SlabShardedLayer, mode_counts, shard_weights
    chunks = torch.arange(2 * 1 * 2 * 3, dtype=torch.float32).reshape(2, 1, 2, 3)   # [world, B, C, cnt]
    full = SlabShardedLayer.assemble(chunks)
    assert full.shape == (1, 2, 6)
    assert full[0, 0].tolist() == [0, 1, 2, 6, 7, 8] and full[0, 1].tolist() == [3, 4, 5, 9, 10, 11]
    assert mode_counts((8, 6, 10), (2, 3, 3)) == ((4, 6, 3), 72)
    W = torch.arange(2 * 2 * 8).reshape(2, 2, 8)
    assert shard_weights(W, 4, 3)[0, 0].tolist() == [6, 7]
    with pytest.raises(ValueError):
        shard_weights(W, 3, 0)
    with pytest.raises(ValueError):
        SlabShardedLayer((9, 4), (2, 2), 1, 1, 1, 2, 0, ops=object())     # 2 does not divide N_0 = 9
    with pytest.raises(ValueError):
        SlabShardedLayer((6, 4), (1, 1), 1, 1, 1, 3, 0, ops=object())     # 3 does not divide M = 2
