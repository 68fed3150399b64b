"""The N > 1 path on CPU: two gloo ranks each take their replica block; together they reproduce
the single-rank schedule bit for bit (the replica id is in the random streams' counters), and the
reported time is the slowest rank's."""
import os
import socket
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, R, J, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import core
    from paper_2003_10579_b200 import sharding
    base, cnt = sharding.split_replicas(rank, world, R)
    tr = core.BulkSchedule("kbatchasync", 8, 3, "shifted_exp", 1.0, 0.5, 7, cnt, replica_base=base).run(J)
    # the product's trace gather (rank-ordered concatenation, uneven blocks, unsigned 16- and 32-bit arrays): every rank
    # hands in tensors shaped like Simulation.trace() and gets the arrays of all replicas
    import torch
    mine = {"t": torch.from_numpy(tr["t"]), "worker": torch.from_numpy(tr["worker"]), "stale": torch.from_numpy(tr["stale"]),
            "K": torch.from_numpy(tr["K"])}
    whole = sharding.gather_traces(mine)
    gathered = [None] * world
    dist.all_gather_object(gathered, (base, cnt))
    slowest = sharding.max_over_ranks(10.0 + rank)
    wb, wc = sharding.replica_block(rank, world, 5)
    np.savez(os.path.join(out_dir, "g%d.npz" % rank), t=whole["t"].numpy(), worker=whole["worker"].numpy(),
             stale=whole["stale"].numpy(), K=whole["K"].numpy(), slowest=slowest,
             bases=np.array([g[0] for g in gathered]), counts=np.array([g[1] for g in gathered]), wb=wb, wc=wc)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_rank_schedule(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    R, J, world = 11, 40, 2
    mp.spawn(_worker, args=(world, port, R, J, str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import core
    full = core.BulkSchedule("kbatchasync", 8, 3, "shifted_exp", 1.0, 0.5, 7, R).run(J)
    for rank in range(world):           # every rank holds the whole trace after the gather
        g = np.load(tmp_path / ("g%d.npz" % rank))
        assert g["bases"].tolist() == [0, 6] and g["counts"].tolist() == [6, 5]
        assert np.array_equal(g["t"].view(np.int64), full["t"].view(np.int64))
        for k in ("worker", "stale", "K"):
            assert g[k].dtype == full[k].dtype and np.array_equal(g[k], full[k]), k
        assert float(g["slowest"]) == 11.0
    assert (int(g["wb"]), int(g["wc"])) == (1 * 5, 5)


def test_gather_traces_is_the_identity_on_one_rank():
    import torch
    sys.path.insert(0, ROOT)
    from paper_2003_10579_b200 import sharding
    tr = {"t": torch.arange(6, dtype=torch.float64).reshape(3, 2)}
    assert sharding.gather_traces(tr)["t"] is tr["t"]
