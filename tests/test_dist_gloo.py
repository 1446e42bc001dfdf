"""World-size-2 gloo test (CPU) of the multi-rank plumbing bench.py uses: batch sharding with no
overlap, per-rank seeds, max-over-ranks timing and whole-job throughput; and that a rank's block
of the grid (Eq. 18) summed over ranks gives the global spectrum (Eq. 6-7) when the exchange is a
plain all-reduce of the oracle's partial spectra."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(WORLD_SIZE=str(world), RANK=str(rank), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from oracle import dtst_oracle as O
    from paper_2607_14394_b200 import dist as D
    assert D.env_world() == (world, rank, rank)
    assert D.init_process_group("gloo")
    try:
        # 1. sharding of a global batch
        lo, hi = D.batch_shard(5, world, rank)
        owned = torch.zeros(5)
        owned[lo:hi] = 1
        dist.all_reduce(owned)
        assert owned.tolist() == [1.0] * 5          # every sample owned exactly once
        # 2. timing reduction and throughput
        ms = D.max_over_ranks([10.0 + rank, 1.0 - rank])
        assert ms == [10.0 + world - 1, 1.0]
        assert D.sum_over_ranks(rank + 1.0) == world * (world + 1) / 2
        assert abs(D.whole_job_throughput(1000.0, ms[0], world) - world * 1000.0 / (ms[0] * 1e-3)) < 1e-6
        assert D.rank_seed(7, rank) != D.rank_seed(7, (rank + 1) % world)
        # 3. DTST over real ranks: slab partial spectra + all-reduce == global spectrum
        N, k = (8, 6, 10), (2, 3, 3)
        x = np.random.default_rng(3).standard_normal((1, 2) + N)
        nl = N[0] // world
        part = O.forward(x[:, :, rank * nl:(rank + 1) * nl], k, N_global=N, offsets=(rank * nl, 0, 0))
        t = torch.view_as_real(torch.from_numpy(np.ascontiguousarray(part)))
        dist.all_reduce(t)
        full = O.forward(x, k)
        err = O.rel_l2(torch.view_as_complex(t).numpy(), full)
        assert err < 1e-12, err
        q.put((rank, "ok"))
    except Exception as e:   # pragma: no cover
        q.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_world_size_2_gloo():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
    assert sorted(results) == [(0, "ok"), (1, "ok")], results


def test_batch_shard_edges():
    from paper_2607_14394_b200 import dist as D
    assert D.batch_shard(1, 4, 0) == (0, 1)
    assert D.batch_shard(1, 4, 3) == (1, 1)          # empty shard
    assert [D.batch_shard(10, 3, r) for r in range(3)] == [(0, 4), (4, 7), (7, 10)]
    with pytest.raises(ValueError):
        D.batch_shard(4, 2, 2)
