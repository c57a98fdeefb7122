"""The N > 1 path on CPU: two gloo ranks shard a batch by candidate range, draw their own
candidates, evaluate them with the oracle, and the pieces equal the unsharded batch; the timing
reduction is a MAX over ranks."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2503_09357_b200.sharding import shard_range, weak_scaling_first


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, K, out_dir):
    import torch.distributed as dist
    from oracle import pe_oracle as orc
    from paper_2503_09357_b200 import workloads as wl
    from paper_2503_09357_b200.sharding import max_over_ranks
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = wl.make_config(1)
    first, count = shard_range(K, world, rank)
    assign, order = wl.make_candidates(w, K=count, first=first)
    res = orc.evaluate(w, assign, order)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), first=first, count=count, makespan=res["makespan"],
             finish=res["finish"], order=order)
    slowest = max_over_ranks(10.0 + rank)            # rank r "measured" 10 + r
    assert slowest == 10.0 + (world - 1)
    dist.barrier()
    dist.destroy_process_group()


def test_shard_range_partitions_exactly():
    for K in (0, 1, 7, 1024, 65537):
        for world in (1, 2, 3, 8):
            pieces = [shard_range(K, world, r) for r in range(world)]
            assert pieces[0][0] == 0 and sum(c for _, c in pieces) == K
            for (f0, c0), (f1, _) in zip(pieces[:-1], pieces[1:]):
                assert f0 + c0 == f1
            assert max(c for _, c in pieces) - min(c for _, c in pieces) <= 1
    assert weak_scaling_first(4096, 3) == 12288


def test_two_gloo_ranks_reproduce_the_unsharded_batch(tmp_path):
    from oracle import pe_oracle as orc
    from paper_2503_09357_b200 import workloads as wl
    K, world = 301, 2
    mp.spawn(_worker, args=(world, _free_port(), K, str(tmp_path)), nprocs=world, join=True)
    w = wl.make_config(1)
    assign, order = wl.make_candidates(w, K=K)
    ref = orc.evaluate(w, assign, order)
    seen = 0
    for r in range(world):
        d = np.load(tmp_path / f"rank{r}.npz")
        f, c = int(d["first"]), int(d["count"])
        assert np.array_equal(d["order"], order[:, f:f + c])
        assert np.array_equal(d["makespan"], ref["makespan"][f:f + c])
        assert np.array_equal(d["finish"], ref["finish"][:, f:f + c])
        seen += c
    assert seen == K
