"""A basis fit whose stored gradients are spread over several processes (one GPU each).

Plumbing only.  Section 2 of the paper has every node compute the covariance of the samples and decompose it;
with the samples sharded over participants the covariance is assembled from additive moments taken about one
common centre per layer:

    rank 0 picks the centre (gvq_fit_centre) ........................ broadcast, n_layers * d floats
    every rank: moments of its own stored gradients (gvq_fit_moments)  one all-reduce (SUM) of
                                                                       n_layers * (1 + d + d * d) doubles
    every rank: the fit from the summed moments (gvq_fit_from_moments) redundantly, as the paper's nodes do

The arithmetic is behind a *fit engine* (the CUDA library here; the tests drive the same plumbing with an engine
made of oracle steps over gloo).
"""
from __future__ import annotations

import torch

from . import gvq


class CudaFitEngine:
    """The three calls of the C ABI on one context."""

    def __init__(self, ctx: "gvq.Context"):
        self.ctx = ctx
        self.device = f"cuda:{ctx.device}"

    def new_centre(self) -> torch.Tensor:
        return torch.zeros((self.ctx.n_layers, self.ctx.d), dtype=torch.float32, device=self.device)

    def new_moments(self) -> torch.Tensor:
        return torch.zeros(self.ctx.layout.fit_moments_count(), dtype=torch.float64, device=self.device)

    def centre(self, hist, centre):
        self.ctx.fit_centre(hist, centre)

    def moments(self, hist, centre, moments):
        self.ctx.fit_moments(hist, centre, moments)

    def finish(self, moments, centre, N, samples_are_sums_of, Ut, mu, evals):
        return self.ctx.fit_from_moments(moments, centre, N, samples_are_sums_of, Ut, mu, evals)


def fit_sharded(engine, hist_local, N: int, samples_are_sums_of: int, Ut, mu, evals, group=None):
    """The fit over all ranks' stored gradients; hist_local: this rank's [L_local][M].  Every rank ends with the same
    (Ut, mu, evals).  Without a process group (or with a single rank) this is the one-GPU fit by way of moments."""
    import torch.distributed as dist
    many = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    centre, moments = engine.new_centre(), engine.new_moments()
    if not many or dist.get_rank(group) == 0:
        engine.centre(hist_local, centre)
    if many:
        src = dist.get_global_rank(group, 0) if group is not None else 0
        dist.broadcast(centre, src=src, group=group)
    engine.moments(hist_local, centre, moments)
    if many:
        dist.all_reduce(moments, group=group)
    return engine.finish(moments, centre, N, samples_are_sums_of, Ut, mu, evals)
