"""The N > 1 path on CPU: two gloo ranks run as independent replicas, only the timing is reduced."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1811_03617_b200 import replicas, workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import oracle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.tiny()
        ids = replicas.rank_node_ids(rank, w.N)
        g = [W.node_gradient(w, n).numpy() for n in ids]
        Ut_t, mu_t = W.random_basis(w)
        s_sum, g_hat = oracle.pipeline(w, g, Ut_t.numpy(), mu_t.numpy())     # the replica's own result
        local_ms = 1.0 + rank                                                 # rank 1 is the slow one
        value, ms = replicas.job_throughput(w.N * w.M * 4, local_ms, world, dist)
        gathered = [None] * world
        dist.all_gather_object(gathered, ids)
        np.save(os.path.join(out_dir, f"g_hat_{rank}.npy"), g_hat)
        if rank == 0:
            np.save(os.path.join(out_dir, "summary.npy"), np.array([value, ms, len({i for l in gathered for i in l})]))
    finally:
        dist.destroy_process_group()


def test_two_replicas_over_gloo(tmp_path, oracle):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    w = W.tiny()
    value, ms, distinct = np.load(tmp_path / "summary.npy")
    assert ms == 2.0                                            # max over ranks, not the mean
    assert np.isclose(value, world * w.N * w.M * 4 / 2.0e-3 / 1e9)
    assert distinct == world * w.N                              # disjoint batches
    # each replica computed exactly what a single process computes for that batch
    Ut_t, mu_t = W.random_basis(w)
    for rank in range(world):
        g = [W.node_gradient(w, n).numpy() for n in replicas.rank_node_ids(rank, w.N)]
        _, want = oracle.pipeline(w, g, Ut_t.numpy(), mu_t.numpy())
        assert np.array_equal(np.load(tmp_path / f"g_hat_{rank}.npy"), want)
    assert not np.array_equal(np.load(tmp_path / "g_hat_0.npy"), np.load(tmp_path / "g_hat_1.npy"))


def test_max_over_ranks_without_a_group():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.rank_node_ids(2, 4) == [8, 9, 10, 11]
