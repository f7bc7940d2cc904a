"""The plumbing of a basis fit spread over ranks (centre broadcast, one all-reduce of the moments, every rank
finishes), run as gloo ranks on CPU with an engine made of the oracle's steps, against the oracle's fit of all
samples at once."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1811_03617_b200 import workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _case():
    w = W.custom("shfit", 160, d=16, k=4, N=4, L=6, layer_len=[16 * 37 + 4, 8, 16 * 90])
    return w, W.stored_gradients(w)


class OracleFitEngine:
    """The fit engine's interface over the oracle (tests only)."""

    def __init__(self, oracle, w):
        self.o, self.w = oracle, w

    def new_centre(self):
        return torch.zeros((self.w.n_layers, self.w.d), dtype=torch.float32)

    def new_moments(self):
        return torch.zeros(self.w.n_layers * (1 + self.w.d + self.w.d ** 2), dtype=torch.float64)

    def centre(self, hist, centre):
        # any point near the mean serves: the first slice of every layer in the first stored gradient
        for l, (o, m) in enumerate(zip(self.w.layer_off, self.w.layer_len)):
            if m >= self.w.d:
                centre[l] = hist[0, o:o + self.w.d]

    def moments(self, hist, centre, moments):
        moments.copy_(torch.from_numpy(self.o.fit_moments(self.w, hist.numpy(), centre.numpy()).ravel()))

    def finish(self, moments, centre, N, c, Ut, mu, evals):
        m = moments.numpy().reshape(self.w.n_layers, -1)
        U, u, e = self.o.fit_from_moments(self.w, m, centre.numpy(), N, c)
        Ut.copy_(torch.from_numpy(U)); mu.copy_(torch.from_numpy(u)); evals.copy_(torch.from_numpy(e))
        return [0] * self.w.n_layers


def _worker(rank, world, port, out_dir):
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    sys.path.insert(0, os.path.dirname(here))
    sys.path.insert(0, here)
    import oracle
    from paper_1811_03617_b200 import sharded_fit
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w, hist = _case()
        mine = hist[rank::world].contiguous()          # the stored gradients this rank holds
        Ut = torch.zeros((w.n_layers, w.k, w.d), dtype=torch.float64)
        mu = torch.zeros((w.n_layers, w.d), dtype=torch.float64)
        ev = torch.zeros((w.n_layers, w.d), dtype=torch.float64)
        sharded_fit.fit_sharded(OracleFitEngine(oracle, w), mine, w.N, w.N, Ut, mu, ev)
        np.savez(os.path.join(out_dir, f"fit_{rank}.npz"), Ut=Ut.numpy(), mu=mu.numpy(), ev=ev.numpy())
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_fit_over_gloo(tmp_path, oracle, world):
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    w, hist = _case()
    o_Ut, o_mu, o_ev, _ = oracle.fit_basis(w, hist.numpy(), N=w.N, samples_are_sums_of=w.N)
    first = None
    for rank in range(world):
        got = np.load(tmp_path / f"fit_{rank}.npz")
        assert np.abs(got["ev"] - o_ev).max() <= 1e-9 * o_ev.max()
        assert np.abs(got["mu"] - o_mu).max() <= 1e-9 * np.abs(o_mu).max()
        for l in range(w.n_layers):
            P = got["Ut"][l] - (got["Ut"][l] @ o_Ut[l].T) @ o_Ut[l]
            assert np.linalg.norm(P, 2) <= 1e-7
        if first is None:
            first = got
        else:   # every rank holds the same result, bit for bit (the same summed moments, the same arithmetic)
            assert all(np.array_equal(got[k], first[k]) for k in ("Ut", "mu", "ev"))


def test_sharded_fit_without_a_process_group(oracle):
    from paper_1811_03617_b200 import sharded_fit
    w, hist = _case()
    Ut = torch.zeros((w.n_layers, w.k, w.d), dtype=torch.float64)
    mu = torch.zeros((w.n_layers, w.d), dtype=torch.float64)
    ev = torch.zeros((w.n_layers, w.d), dtype=torch.float64)
    sharded_fit.fit_sharded(OracleFitEngine(oracle, w), hist, w.N, w.N, Ut, mu, ev)
    _, o_mu, o_ev, _ = oracle.fit_basis(w, hist.numpy(), N=w.N, samples_are_sums_of=w.N)
    assert np.abs(ev.numpy() - o_ev).max() <= 1e-9 * o_ev.max() and np.abs(mu.numpy() - o_mu).max() <= 1e-9 * np.abs(o_mu).max()
