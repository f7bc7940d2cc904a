"""Algorithm 1's plumbing on CPU: the participants of ``paper_1811_03617_b200.ring`` driven by an engine made of
the oracle's steps, stepped in one process and run as gloo ranks, against the direct evaluation of Eq. 3-5."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1811_03617_b200 import ring, workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case(world, n_local):
    w = W.custom("ring", 140 + world, d=16, k=4, N=world * n_local, L=1,
                 layer_len=[16 * 7 + 4, 8, 16 * 30, 16 * 3 + 4, 0, 16 * 11, 12])
    g = W.node_gradients(w)
    Ut, mu = W.random_basis(w)
    return w, g, Ut, mu


@pytest.mark.parametrize("world,n_local", [(1, 2), (2, 1), (3, 2), (4, 1), (7, 1)])
def test_local_ring_follows_algorithm_1(oracle, world, n_local):
    from ring_engine import OracleSegmentEngine
    w, g, Ut, mu = _case(world, n_local)
    lr = ring.LocalRing(lambda: OracleSegmentEngine(oracle, w, world), world)
    g_hat = [torch.zeros(w.M, dtype=torch.float64) for _ in range(world)]
    lr.run([g[n * n_local:(n + 1) * n_local] for n in range(world)], w.N, Ut, mu, g_hat)
    _, want = oracle.pipeline(w, [x.numpy() for x in g], Ut.numpy(), mu.numpy())
    for n in range(world):
        assert np.abs(g_hat[n].numpy() - want).max() <= 1e-12 * np.abs(want).max()
    # the same messages as the oracle's node-by-node simulation of Algorithm 1 (sizes per node)
    if n_local == 1:
        _, sent = oracle.ring_allreduce(w, [x.numpy() for x in g], Ut.numpy(), mu.numpy())
        assert [p.floats_sent for p in lr.nodes] == sent
    assert sum(p.floats_sent for p in lr.nodes) == 2 * (world - 1) * (w.S * w.k + w.tail_entries)


def _worker(rank, world, n_local, port, out_dir):
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    sys.path.insert(0, os.path.dirname(here))
    sys.path.insert(0, here)
    import oracle
    from ring_engine import OracleSegmentEngine
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w, g, Ut, mu = _case(world, n_local)
        p = ring.RingParticipant(OracleSegmentEngine(oracle, w, world), ring.DistTransport())
        g_hat = torch.zeros(w.M, dtype=torch.float64)
        p.run(g[rank * n_local:(rank + 1) * n_local], w.N, Ut, mu, g_hat)
        np.save(os.path.join(out_dir, f"g_hat_{rank}.npy"), g_hat.numpy())
        np.save(os.path.join(out_dir, f"sent_{rank}.npy"), np.array([p.floats_sent]))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,n_local", [(2, 1), (3, 2)])
def test_ring_over_gloo(tmp_path, oracle, world, n_local):
    port = _free_port()
    mp.spawn(_worker, args=(world, n_local, port, str(tmp_path)), nprocs=world, join=True)
    w, g, Ut, mu = _case(world, n_local)
    _, want = oracle.pipeline(w, [x.numpy() for x in g], Ut.numpy(), mu.numpy())
    sent = 0
    for rank in range(world):
        got = np.load(tmp_path / f"g_hat_{rank}.npy")
        assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
        sent += int(np.load(tmp_path / f"sent_{rank}.npy")[0])
    assert sent == 2 * (world - 1) * (w.S * w.k + w.tail_entries)


def _collective_worker(rank, world, n_local, port, out_dir):
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    sys.path.insert(0, os.path.dirname(here))
    sys.path.insert(0, here)
    import oracle
    from ring_engine import OracleSegmentEngine
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w, g, Ut, mu = _case(world, n_local)
        engine = OracleSegmentEngine(oracle, w, 1)
        x = engine.new_buffer(engine.x_floats[0])
        g_hat = torch.zeros(w.M, dtype=torch.float64)
        ring.allreduce_compressed(engine, g[rank * n_local:(rank + 1) * n_local], w.N, Ut, mu, x, g_hat)
        np.save(os.path.join(out_dir, f"g_hat_{rank}.npy"), g_hat.numpy())
        np.save(os.path.join(out_dir, f"x_{rank}.npy"), x[: engine.x_floats[0]].numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,n_local", [(2, 1), (3, 2)])
def test_one_collective_of_the_compressed_buffer_over_gloo(tmp_path, oracle, world, n_local):
    """The by-node partition of the job: every rank compresses its own nodes' gradients with the job's N, ONE
    all-reduce carries the exchange buffer (S k + T floats instead of M), every rank decompresses."""
    port = _free_port()
    mp.spawn(_collective_worker, args=(world, n_local, port, str(tmp_path)), nprocs=world, join=True)
    w, g, Ut, mu = _case(world, n_local)
    s_want, want = oracle.pipeline(w, [x.numpy() for x in g], Ut.numpy(), mu.numpy())
    for rank in range(world):
        got = np.load(tmp_path / f"g_hat_{rank}.npy")
        assert np.abs(got - want).max() <= 1e-12 * np.abs(want).max()
        x = np.load(tmp_path / f"x_{rank}.npy")
        assert x.size == w.S * w.k + w.tail_entries                    # what crossed the link: k / d of the gradient
        assert np.abs(x[: w.S * w.k] - s_want.ravel()).max() <= 1e-12 * np.abs(s_want).max()


def test_one_collective_without_a_process_group(oracle):
    """World 1: no collective at all, the result is the one-process path."""
    from ring_engine import OracleSegmentEngine
    w, g, Ut, mu = _case(1, 3)
    engine = OracleSegmentEngine(oracle, w, 1)
    x = engine.new_buffer(engine.x_floats[0])
    g_hat = torch.zeros(w.M, dtype=torch.float64)
    ring.allreduce_compressed(engine, g, w.N, Ut, mu, x, g_hat)
    _, want = oracle.pipeline(w, [t.numpy() for t in g], Ut.numpy(), mu.numpy())
    assert np.abs(g_hat.numpy() - want).max() <= 1e-12 * np.abs(want).max()
    with pytest.raises(ValueError):
        ring.allreduce_compressed(OracleSegmentEngine(oracle, w, 2), g, w.N, Ut, mu, x, g_hat)


def test_segment_layouts_agree_with_the_oracle(oracle):
    """gvq_segment_layout (host helper of the C ABI) against the oracle's reading of "N equal segments"."""
    from paper_1811_03617_b200 import gvq
    cases = [(W.custom("s", 150, d=16, k=4, N=1, L=1, layer_len=[16 * 7 + 4, 8, 16 * 30, 16 * 3 + 4, 0, 16 * 11, 12]), G)
             for G in (1, 2, 3, 4, 7, 64)] + [(W.resnet50(), 16), (W.resnet32(), 8), (W.vgg16(), 5)]
    for w, G in cases:
        hl = gvq.HostLayout.of(w)
        assert hl.exchange_floats() == w.S * w.k + w.tail_entries
        total = 0
        for j in range(G):
            seg, layers = gvq.segment_layout(hl, G, j)
            want = oracle.segment_layout(w, G, j)
            if seg is None:
                assert want.n_layers == 0
                continue
            assert seg.layer_off == want.layer_off and seg.layer_len == want.layer_len
            assert layers == want.piece_layer
            assert seg.check() == 0
            total += seg.exchange_floats()
        assert total == hl.exchange_floats()


def test_segment_layout_refuses_bad_arguments():
    import ctypes
    from paper_1811_03617_b200 import gvq
    hl = gvq.HostLayout.of(W.tiny())
    n = ctypes.c_int32(0)
    lay = (ctypes.c_int32 * 1)()
    off, ln = (ctypes.c_int64 * 1)(), (ctypes.c_int64 * 1)()
    L = gvq.lib()
    assert L.gvq_segment_layout(ctypes.byref(hl.c), 0, 0, ctypes.byref(n), lay, off, ln) == 2      # no segments
    assert L.gvq_segment_layout(ctypes.byref(hl.c), 4, 4, ctypes.byref(n), lay, off, ln) == 2      # j out of range
    assert L.gvq_segment_layout(ctypes.byref(hl.c), 4, 0, None, lay, off, ln) == 1
    assert L.gvq_segment_layout(None, 4, 0, ctypes.byref(n), lay, off, ln) == 1
    assert L.gvq_exchange_floats(None) == -1
    assert L.gvq_segment_layout(ctypes.byref(hl.c), 4, 3, ctypes.byref(n), lay, off, ln) == 0
    assert n.value == 1 and off[0] == 3 * 256 * 16 and ln[0] == 256 * 16     # the last quarter of the single layer
