"""A segment engine for the ring plumbing made of the oracle's fp64 CPU steps (tests only): the schedule and the
transports of ``paper_1811_03617_b200.ring`` can then run on CPU tensors, over gloo or in one process."""
import numpy as np
import torch


class OracleSegmentEngine:
    def __init__(self, oracle, layout, n_segments: int):
        self.o, self.layout, self.n_segments = oracle, layout, int(n_segments)
        self.segs = [oracle.segment_layout(layout, n_segments, j) for j in range(n_segments)]
        self.x_floats = [(sg.slice1 - sg.slice0) * int(layout.k) + sum(m % sg.d for m in sg.layer_len) for sg in self.segs]

    def new_buffer(self, n_floats):
        return torch.zeros(max(n_floats, 4), dtype=torch.float64)

    def _basis(self, j, Ut, mu):
        return self.o._segment_basis(self.layout, self.segs[j], Ut.numpy(), mu.numpy())

    def compress(self, j, g_local, N, Ut, mu, x):
        sg = self.segs[j]
        if sg.n_layers == 0:
            return
        U, m = self._basis(j, Ut, mu)
        s = sum(self.o.compress(sg, g.numpy(), U, m, N) for g in g_local)
        t = sum(self.o._segment_tails(sg, g.numpy()) for g in g_local)
        x[: self.x_floats[j]] = torch.from_numpy(np.concatenate([s.ravel(), t]))

    def accumulate(self, j, x_acc, x_in):
        x_acc += x_in

    def decompress(self, j, x, Ut, mu, g_hat):
        sg = self.segs[j]
        if sg.n_layers == 0:
            return
        U, m = self._basis(j, Ut, mu)
        nS = sg.slice1 - sg.slice0
        xs = x[: self.x_floats[j]].numpy()
        s, t = xs[: nS * sg.k].reshape(nS, sg.k), xs[nS * sg.k:]
        whole = self.o.SegmentLayout(sg.d, sg.k, sg.piece_layer, sg.layer_off, [(q // sg.d) * sg.d for q in sg.layer_len],
                                     sg.slice0, sg.slice1)
        part = self.o.decompress(whole, s, U, m, None, 1, g_hat.numel())
        out = g_hat.numpy()
        p = 0
        for o, q in zip(sg.layer_off, sg.layer_len):
            full = (q // sg.d) * sg.d
            out[o:o + full] = part[o:o + full]
            out[o + full:o + q] = t[p:p + q - full]
            p += q - full
