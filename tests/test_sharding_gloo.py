"""The N > 1 path on CPU: two gloo ranks shard the heads of a workload with no data-path collective;
the union of what they own is the whole workload, and the timing reduction (max over ranks) works."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2407_13885_b200 import inputs


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    w = inputs.Workload("t", "fused", B=1, H=5, N=24, d=16, scale=0.25, cfg_id=7)
    begin, end, seed = inputs.rank_heads(w, rank, world, "strong")   # the function bench.py --scaling strong uses
    assert (begin, end) == inputs.shard_range(w.B * w.H, rank, world) and seed == inputs.SEED
    q, k = inputs.make_qk(w, begin, end, seed=seed)            # only this rank's heads are drawn
    P = oracle.attnw(q.reshape(1, end - begin, w.N, w.d), k.reshape(1, end - begin, w.N, w.d), w.scale)
    np.save(os.path.join(out_dir, f"p{rank}.npy"), P)
    # what bench.py does with its timings and launch counts
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    n = torch.tensor([end - begin], dtype=torch.int64)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    assert t.item() == 10.0 + world - 1 and n.item() == w.B * w.H
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_cover_the_workload(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    import oracle
    w = inputs.Workload("t", "fused", B=1, H=5, N=24, d=16, scale=0.25, cfg_id=7)
    q, k = inputs.make_qk(w)
    full = oracle.attnw(q.reshape(1, 5, w.N, w.d), k.reshape(1, 5, w.N, w.d), w.scale)
    parts = [np.load(os.path.join(str(tmp_path), f"p{r}.npy")) for r in range(world)]
    assert [p.shape[1] for p in parts] == [3, 2]                 # remainder goes to the first rank
    assert np.array_equal(np.concatenate(parts, axis=1), full)


def test_rank_heads_uneven_splits_and_weak_replicas():
    w5 = inputs.Workload("t", "fused", B=1, H=5, N=24, d=16, scale=0.25, cfg_id=7)
    assert [inputs.rank_heads(w5, r, 2, "strong")[:2] for r in range(2)] == [(0, 3), (3, 5)]
    c3 = inputs.WORKLOADS["c3"]                                   # 128 heads over 3 ranks: 43 + 43 + 42
    parts = [inputs.rank_heads(c3, r, 3, "strong")[:2] for r in range(3)]
    assert parts == [(0, 43), (43, 86), (86, 128)]
    for world in (1, 2, 3, 4, 7, 8, 128, 200):                    # contiguous, disjoint, complete; empty ranks allowed
        cuts = [inputs.rank_heads(c3, r, world, "strong")[:2] for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == 128
        assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
        sizes = [e - b for b, e in cuts]
        assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    # weak scaling: every rank owns a whole replica, drawn with its own seed
    assert inputs.rank_heads(c3, 2, 4, "weak") == (0, 128, inputs.SEED + 2)
