"""The multi-rank path on CPU: two gloo ranks partition the problems, each ranks its block
(the oracle stands in for the GPU call), the blocks are all-gathered, and the result equals
the unsharded ranking. Also the MAX reduction used for timing."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_35587_b200 import sharding


def test_partition_covers_every_problem_once():
    for P in (0, 1, 2, 7, 1024, 4097):
        for world in (1, 2, 3, 8):
            parts = sharding.partition(P, world)
            assert len(parts) == world and parts[0][0] == 0 and parts[-1][1] == P
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, P, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2609_35587_b200 import workloads as wl
    oracle.set_threads(1)
    w = wl.make_workload(0, P=P, C=300, trees=8, depth=4)

    def select_fn(block):
        idx, sc = oracle.select(block, w.candidates, w.desc, w.k, gbdt=w.gbdt)
        return torch.from_numpy(idx), torch.from_numpy(sc)

    idx, sc = sharding.select_sharded(select_fn, w.problems, w.k, torch.device("cpu"))
    t = sharding.max_over_ranks(10.0 + rank, torch.device("cpu"))

    # candidate split of the single-problem call: each rank ranks its share of the pool, the
    # world x k pairs are gathered and merged (the oracle's top-k stands in for ks_merge_topk)
    def select_part(lo, hi):
        pool = np.arange(lo, hi, dtype=np.int32)
        i1, s1 = oracle.select(w.problems[:1], w.candidates, w.desc, w.k, gbdt=w.gbdt,
                               seg_off=np.array([0, hi - lo], np.int64), seg_idx=pool)
        return torch.from_numpy(i1[0]), torch.from_numpy(s1[0])

    def merge(i_all, s_all, k):
        live = np.nonzero(i_all.numpy()[0] >= 0)[0]
        mi, ms = oracle.topk(s_all.numpy()[0][live], 1, k, seg_off=np.array([0, len(live)], np.int64),
                             seg_idx=i_all.numpy()[0][live].astype(np.int32))
        return torch.from_numpy(mi), torch.from_numpy(ms)

    one_i, one_s = [], []
    for C in (300, 1):   # the second: a rank with no candidates at all
        oi, os_ = sharding.select_one_sharded(select_part, merge, C, w.k, torch.device("cpu"))
        one_i.append(oi.numpy())
        one_s.append(os_.numpy())
    if rank == 0:
        q.put((idx.numpy(), sc.numpy(), t, one_i, one_s))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_match_the_unsharded_ranking():
    import oracle
    from paper_2609_35587_b200 import workloads as wl
    for P in (7, 1):  # odd split, and a rank with no problems at all
        ctx = mp.get_context("spawn")
        q = ctx.Queue()
        port = _free_port()
        procs = [ctx.Process(target=_worker, args=(r, 2, port, P, q)) for r in range(2)]
        for p in procs:
            p.start()
        idx, sc, t, one_i, one_s = q.get(timeout=120)
        for p in procs:
            p.join(timeout=120)
            assert p.exitcode == 0
        w = wl.make_workload(0, P=P, C=300, trees=8, depth=4)
        ridx, rsc = oracle.select(w.problems, w.candidates, w.desc, w.k, gbdt=w.gbdt)
        assert np.array_equal(idx, ridx) and np.array_equal(sc, rsc)
        assert t == 11.0
        for C, oi, os_ in zip((300, 1), one_i, one_s):
            r1i, r1s = oracle.select(w.problems[:1], w.candidates[:C], w.desc, w.k, gbdt=w.gbdt)
            assert np.array_equal(oi, r1i[0]) and np.array_equal(os_, r1s[0])
