"""Multi-rank host logic on CPU (gloo, world_size 2): heads are sharded with no data-path
collective, each rank's shard equals the corresponding slice of the unsharded result, and
the timing reduction is a max over ranks.  The per-rank compute is stood in for by the
fp64 oracle (this is a test; the product path has no CPU route)."""
import os
import socket

import numpy as np
import pytest

from paper_2609_33916_b200 import sharding


def test_head_shard_partitions():
    for total in (1, 5, 16, 17, 32):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                s, c = sharding.head_shard(total, world, r)
                seen.extend(range(s, s + c))
            assert seen == list(range(total))
    assert sharding.head_shard(16, 8, 3) == (6, 2)
    with pytest.raises(ValueError):
        sharding.head_shard(4, 2, 2)
    assert sharding.aggregate_rate([10.0, 10.0], [1.0, 2.0]) == 10.0


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    B, H, n, d = 1, 5, 48, 8
    rng = np.random.default_rng(0)   # same seed on every rank: every rank can slice the same global problem
    Q, K, V, dO = (rng.standard_normal((B, H, n, d)) for _ in range(4))
    s, c = sharding.head_shard(B * H, world, rank)
    sl = slice(s, s + c)
    mine = oracle.attn_fwd_bwd(Q[:, sl], K[:, sl], V[:, sl], dO[:, sl], True, 0.3)
    # timing reduction: max over ranks
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert float(t) == float(world)
    dist.barrier()
    np.save(os.path.join(out_dir, f"dq_{rank}.npy"), mine["dQ"])
    np.save(os.path.join(out_dir, f"o_{rank}.npy"), mine["O"])
    dist.barrier()
    if rank == 0:
        full = oracle.attn_fwd_bwd(Q, K, V, dO, True, 0.3)
        got_dq = np.concatenate([np.load(os.path.join(out_dir, f"dq_{r}.npy")) for r in range(world)], axis=1)
        got_o = np.concatenate([np.load(os.path.join(out_dir, f"o_{r}.npy")) for r in range(world)], axis=1)
        np.testing.assert_array_equal(got_dq, full["dQ"])
        np.testing.assert_array_equal(got_o, full["O"])
    dist.destroy_process_group()


def test_two_rank_head_sharding_gloo(tmp_path):
    import torch.multiprocessing as mp
    mp.spawn(_worker, args=(2, _free_port(), str(tmp_path)), nprocs=2, join=True)
