"""gvq_fit_basis_static: the basis fit for callers that cannot allocate device memory.

Some users of this library run inside a host application that has already handed all device memory
to its own allocator, or that bans cudaMalloc on the training thread because it can stall the whole
device.  They have no workspace to give gvq_fit_basis, so the library offers the same fit on a fixed
scratch array that lives in the library image.  This file checks, through the C ABI, that the
entry point returns what gvq_fit_basis returns, on two calls in a row (the array keeps the previous
call's contents, so the second call must not be disturbed by the first), and that it refuses a
layout whose fit would not fit the array.  It is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_1811_03617_b200 import workloads as W
from util import subspace_angle

pytestmark = pytest.mark.gpu


def _fit(ctx, w, hist, static):
    Ut = torch.full((w.n_layers, w.k, w.d), float("nan"), device="cuda")
    mu = torch.full((w.n_layers, w.d), float("nan"), device="cuda")
    ev = torch.full((w.n_layers, w.d), float("nan"), device="cuda")
    sweeps = (ctx.fit_basis_static if static else ctx.fit_basis)(hist, w.N, w.N, Ut, mu, ev)
    return Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), sweeps


def _same_fit(w, got, want):
    Ut_s, mu_s, ev_s, sw_s = got
    Ut_w, mu_w, ev_w, sw_w = want
    assert np.isfinite(Ut_s).all() and np.isfinite(mu_s).all() and np.isfinite(ev_s).all()
    assert sw_s == sw_w
    for l in range(w.n_layers):
        lam_max = max(float(ev_w[l, 0]), 1e-30)
        assert np.abs(ev_s[l] - ev_w[l]).max() <= 1e-5 * lam_max
        assert np.allclose(mu_s[l], mu_w[l], rtol=1e-5, atol=1e-6 * (np.abs(mu_w[l]).max() + 1e-30))
        assert subspace_angle(Ut_s[l], Ut_w[l]) <= 1e-4


def test_static_fit_matches_workspace_fit_twice_in_a_row():
    from paper_1811_03617_b200 import gvq
    w = W.resnet32()
    assert gvq.HostLayout.of(w).fit_workspace_bytes(w.L) <= 4 << 20
    ctx = gvq.Context(w)
    hist_a = W.stored_gradients(w, device="cuda")
    hist_b = W.stored_gradients(w, device="cuda", first_iteration=100)
    want_a = _fit(ctx, w, hist_a, static=False)
    want_b = _fit(ctx, w, hist_b, static=False)
    ctx.set_workspace(None)                      # the static entry point must not need it
    got_a = _fit(ctx, w, hist_a, static=True)    # first call: also looks up the array's address
    got_b = _fit(ctx, w, hist_b, static=True)    # second call: runs on the first call's leftovers
    _same_fit(w, got_a, want_a)
    _same_fit(w, got_b, want_b)
    assert not np.array_equal(got_a[0], got_b[0])  # the two fits really differ
    # a second context on the same device shares the array
    tiny = W.tiny()
    ctx2 = gvq.Context(tiny)
    h = W.stored_gradients(tiny, device="cuda")
    _same_fit(tiny, _fit(ctx2, tiny, h, static=True), _fit(ctx2, tiny, h, static=False))


def test_static_fit_refuses_what_does_not_fit():
    from paper_1811_03617_b200 import gvq
    w = W.resnet50()
    assert gvq.HostLayout.of(w).fit_workspace_bytes(4) > 4 << 20
    ctx = gvq.Context(w)
    hist = torch.zeros((1, w.M), device="cuda")
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda")
    mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    st = gvq.lib().gvq_fit_basis_static(ctx._h, hist.data_ptr(), w.M, 1, w.N, w.N, Ut.data_ptr(), mu.data_ptr(),
                                        ev.data_ptr(), None)
    assert st == 5  # GVQ_ERR_WORKSPACE
    st = gvq.lib().gvq_fit_basis_static(ctx._h, None, w.M, 1, w.N, w.N, Ut.data_ptr(), mu.data_ptr(), ev.data_ptr(), None)
    assert st == 1  # GVQ_ERR_NULL
