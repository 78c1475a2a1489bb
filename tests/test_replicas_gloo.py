"""The multi-GPU bookkeeping (candidate sharding, max-over-ranks timing, record gather) run as two gloo
ranks on CPU. Each rank 'verifies' its shard with the oracle, the gathered records must equal the
single-process result."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, ret):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import gv_oracle as O
    from paper_2507_23194_b200 import replicas as R, workloads as W
    wl = W.config1("cpu", n=5000)
    ref = wl.ref.numpy()

    def verify_local(ref_t, cands):          # the oracle stands in for the CUDA library's dense call on CPU ranks
        recs = O.verify_batch(ref_t.numpy(), [c.numpy() for c in cands], O.F32, wl.atol, wl.rtol, wl.equal_nan)
        return torch.from_numpy(recs.view(np.uint8).reshape(-1, 64).copy())

    # the code path bench.py's candidate-sharded mode takes: plan, local verify, gather
    counts, mine = R.shard_plan(len(wl.cands), world, rank)
    assert mine == R.shard_candidates(len(wl.cands), world, rank) and sum(counts) == len(wl.cands)
    allrec = R.verify_sharded(wl.ref, wl.cands, verify_local, world, rank)
    slowest = R.max_over_ranks(10.0 + rank)
    total = R.aggregate_throughput(1_000_000, slowest)
    if rank == 0:
        want = O.verify_batch(ref, [c.numpy() for c in wl.cands], O.F32, wl.atol, wl.rtol, wl.equal_nan)
        ret["same"] = allrec.numpy().tobytes() == want.tobytes()
        ret["slowest"] = slowest
        ret["total"] = total
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_share_a_batch():
    from oracle import gv_oracle
    gv_oracle.build()
    world = 2
    mgr = mp.Manager()
    ret = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), ret), nprocs=world, join=True)
    assert ret["same"] is True
    assert ret["slowest"] == 11.0
    assert abs(ret["total"] - 2 * 1_000_000 / 11e-3 / 1e9) < 1e-9


def test_shards_partition_the_candidates():
    from paper_2507_23194_b200 import replicas as R
    for n in (0, 1, 7, 8, 255, 256):
        for world in (1, 2, 3, 8):
            got = sum((R.shard_candidates(n, world, r) for r in range(world)), [])
            assert got == list(range(n))
            sizes = [len(R.shard_candidates(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        R.shard_candidates(4, 2, 2)
