"""Failure paths and stream rules of the C ABI on a GPU, none of which faults or hangs the device: the sweep limit of
the eigen-solver (GVQ_ERR_NOT_CONVERGED), a bounded wait inside the tensor-core projection that runs out
(GVQ_ERR_TIMEOUT: the kernel returns, the status word is read and cleared, the context stays usable), a new buffer
met during stream capture (GVQ_ERR_CAPTURE), and a context whose calls alternate between two streams."""
import numpy as np
import pytest
import torch

from paper_1811_03617_b200 import workloads as W
from util import rel_l2

pytestmark = pytest.mark.gpu

NOT_CONVERGED, TIMEOUT, CAPTURE = 7, 9, 10


@pytest.fixture(scope="module")
def gvq():
    from paper_1811_03617_b200 import gvq as _gvq
    _gvq.lib()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return _gvq


def _fit_outputs(w):
    return (torch.full((w.n_layers, w.k, w.d), float("nan"), device="cuda"),
            torch.full((w.n_layers, w.d), float("nan"), device="cuda"),
            torch.full((w.n_layers, w.d), float("nan"), device="cuda"))


@pytest.mark.parametrize("fit_path", [1, 2], ids=["rotations_kept", "values_and_subspace"])
def test_sweep_limit_reports_not_converged_and_the_context_recovers(gvq, oracle, fit_path):
    w = W.custom("sweepcap", 801, d=64, k=8, N=4, L=4, layer_len=[64 * 200, 64 * 90 + 12])
    hist = W.stored_gradients(w)
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut, mu, ev = _fit_outputs(w)
    ctx.set_limits(max_sweeps=1)
    with pytest.raises(gvq.GvqError) as e:
        ctx.fit_basis(hist.cuda(), w.N, w.N, Ut, mu, ev)
    assert e.value.status == NOT_CONVERGED
    # the outputs are written all the same: finite, and the mean does not depend on the solver at all
    assert torch.isfinite(Ut).all() and torch.isfinite(mu).all() and torch.isfinite(ev).all()
    o_Ut, o_mu, o_ev, _ = oracle.fit_basis(w, hist.numpy(), N=w.N, samples_are_sums_of=w.N)
    assert np.allclose(mu.cpu().numpy(), o_mu, rtol=1e-5, atol=1e-6 * np.abs(o_mu).max())
    # back to the default limit: the same context converges and meets the bars
    ctx.set_limits(max_sweeps=0)
    sweeps = ctx.fit_basis(hist.cuda(), w.N, w.N, Ut, mu, ev)
    assert all(1 < s < 30 for s in sweeps)
    for l in range(w.n_layers):
        assert np.abs(ev[l].cpu().numpy()[: w.k] - o_ev[l][: w.k]).max() <= 1e-5 * o_ev[l][0]


def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(gvq, oracle):
    """The projection's first CTA leaves out its last load (a host-side switch), so the wait for it ends at the
    (shortened) limit: the kernel gives up cleanly, gvq_device_status reports it once, the next call is correct."""
    w = W.custom("dropload", 802, d=128, k=16, N=3, L=1, layer_len=[128 * 700 + 40])     # 1 MB per node, 6 tiles
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [torch.as_tensor(x).cuda() for x in g]
    ctx = gvq.Context(w)
    s_sum = torch.zeros((ctx.S, w.k), device="cuda")
    g_hat = torch.zeros(w.M, device="cuda")
    ctx.compress_aggregate(g_dev, Ut, mu, s_sum)          # an ordinary call first
    ctx.device_status()
    want = s_sum.clone()
    ctx.set_limits(wait_cycles=2_000_000)                 # ~1 ms of SM clock
    ctx.test_drop_load(True)
    ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
    with pytest.raises(gvq.GvqError) as e:
        ctx.device_status()
    assert e.value.status == TIMEOUT
    ctx.device_status()                                   # the word was cleared by the report
    ctx.test_drop_load(False)
    ctx.set_limits(wait_cycles=0)
    s_sum.fill_(float("nan"))
    ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
    ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    ctx.device_status()
    assert torch.equal(s_sum, want)
    o_s, o_g = oracle.pipeline(w, g, Ut_t.numpy(), mu_t.numpy())
    assert rel_l2(s_sum.cpu().numpy(), o_s) <= 1e-5 and rel_l2(g_hat.cpu().numpy(), o_g) <= 1e-5


def test_the_decompression_gives_up_cleanly_too(gvq, oracle):
    """The same hook on the decompression: its first CTA's converters do not hand over their first tile, the MMA warp's
    wait for it ends at the shortened limit, every role leaves, the status is reported once and the next call is right."""
    w = W.custom("dropdec", 807, d=128, k=16, N=2, L=1, layer_len=[128 * 700 + 40, 128 * 260])
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [torch.as_tensor(x).cuda() for x in g]
    ctx = gvq.Context(w)
    s_sum = torch.zeros((ctx.S, w.k), device="cuda")
    g_hat = torch.zeros(w.M, device="cuda")
    ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
    ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    ctx.device_status()
    want = g_hat.clone()
    ctx.set_limits(wait_cycles=2_000_000)
    ctx.test_drop_load(True)
    ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    with pytest.raises(gvq.GvqError) as e:
        ctx.device_status()
    assert e.value.status == TIMEOUT
    ctx.test_drop_load(False)
    ctx.set_limits(wait_cycles=0)
    g_hat.fill_(float("nan"))
    ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    ctx.device_status()
    assert torch.equal(g_hat, want)
    _, o_g = oracle.pipeline(w, g, Ut_t.numpy(), mu_t.numpy())
    assert rel_l2(g_hat.cpu().numpy(), o_g) <= 1e-5


def test_the_tensor_core_covariance_gives_up_cleanly_too(gvq, oracle):
    """The covariance kernel's first CTA leaves out its first load: gvq_fit_basis returns GVQ_ERR_TIMEOUT (and clears
    the word itself), the same context then fits correctly."""
    w = W.custom("dropcov", 808, d=128, k=16, N=4, L=3, layer_len=[128 * 600, 128 * 200 + 8])
    hist = W.stored_gradients(w)
    ctx = gvq.Context(w)
    Ut, mu, ev = _fit_outputs(w)
    ctx.set_limits(wait_cycles=2_000_000)
    ctx.test_drop_load(True)
    with pytest.raises(gvq.GvqError) as e:
        ctx.fit_basis(hist.cuda(), w.N, w.N, Ut, mu, ev)
    assert e.value.status == TIMEOUT
    ctx.device_status()                                   # already cleared by the fit entry point
    ctx.test_drop_load(False)
    ctx.set_limits(wait_cycles=0)
    ctx.fit_basis(hist.cuda(), w.N, w.N, Ut, mu, ev)
    o_Ut, o_mu, o_ev, _ = oracle.fit_basis(w, hist.numpy(), N=w.N, samples_are_sums_of=w.N)
    for l in range(w.n_layers):
        assert np.abs(ev[l].cpu().numpy() - o_ev[l]).max() <= 1e-5 * o_ev[l][0]
        G = Ut[l].cpu().numpy().astype(np.float64)
        assert np.linalg.norm(G - (G @ o_Ut[l].T) @ o_Ut[l], 2) <= 1e-4


def test_a_new_buffer_during_capture_is_refused(gvq):
    w = W.custom("capture_new", 803, d=128, k=16, N=2, L=1, layer_len=[128 * 300 + 40, 128 * 129])
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    unseen = [x.clone() for x in g_dev]
    ctx = gvq.Context(w)
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        ctx.compress_aggregate(g_dev, Ut, mu, s_sum)      # these buffers are known to the context now
    torch.cuda.synchronize()
    want = s_sum.clone()
    graph = torch.cuda.CUDAGraph()
    status = None
    with torch.cuda.graph(graph):
        try:
            ctx.compress_aggregate(unseen, Ut, mu, s_sum)
        except gvq.GvqError as exc:
            status = exc.status
        ctx.compress_aggregate(g_dev, Ut, mu, s_sum)      # known buffers are fine inside the same capture
    assert status == CAPTURE
    s_sum.zero_()
    graph.replay()
    torch.cuda.synchronize()
    ctx.device_status()
    assert torch.equal(s_sum, want)
    ctx.compress_aggregate(unseen, Ut, mu, s_sum)         # outside a capture the new buffers are taken
    ctx.device_status()
    assert torch.equal(s_sum, want)


def test_calls_alternating_between_two_streams_stay_ordered(gvq):
    """A context's scratch is ordered by its stream; when the binding hands it another stream the library orders the
    new stream behind the old one.  Steps issued alternately on two streams, without any host synchronisation in
    between, give the result of the same steps on one stream, bit for bit."""
    lens = [256 * 300 + 64, 256 * 129, 256 * 40]
    w = W.custom("two_streams", 804, d=256, k=32, N=5, L=1, layer_len=lens)
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx = gvq.Context(w)
    s = [torch.empty((ctx.S, w.k), device="cuda") for _ in range(2)]
    h = [torch.zeros(w.M, device="cuda") for _ in range(2)]
    ctx.compress_aggregate(g_dev, Ut, mu, s[0])
    ctx.decompress(s[0], Ut, mu, g_dev, w.N, h[0])
    ctx.device_status()
    want_s, want_h = s[0].clone(), h[0].clone()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for st in streams:
        st.wait_stream(torch.cuda.current_stream())
    for rep in range(6):
        i = rep & 1
        with torch.cuda.stream(streams[i]):
            ctx.compress_aggregate(g_dev, Ut, mu, s[i])
            ctx.decompress(s[i], Ut, mu, g_dev, w.N, h[i])
    torch.cuda.synchronize()
    ctx.device_status()
    for i in range(2):
        assert torch.equal(s[i], want_s) and torch.equal(h[i], want_h)


@pytest.mark.parametrize("chunked", [False, True], ids=["one_piece", "chunks"])
def test_allreduce_host_quantized_matches_the_device_calls(gvq, chunked):
    """The host-buffer form of the quantized step: same bits as gvq_compress_quantize_aggregate + gvq_decompress on
    device buffers, in one piece and in chunks (the quantizer is keyed on the slice's index in the whole layout)."""
    if chunked:
        base = W.resnet50()
        w = W.custom("hostq_chunks", 805, d=base.d, k=base.k, N=2, L=1, layer_len=base.layer_len)
    else:
        w = W.custom("hostq", 806, d=128, k=16, N=3, L=1, layer_len=[128 * 300 + 20, 128 * 129])
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx = gvq.Context(w)
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    ctx.compress_quantize_aggregate(g_dev, Ut, mu, 7, 99, s_sum)
    ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    ctx.device_status()
    g_pinned = [x.cpu().pin_memory() for x in g_dev]
    out = torch.full((w.M,), float("nan")).pin_memory()
    if chunked:
        ctx.host_prepare()
    ctx.allreduce_host(g_pinned, Ut, mu, out, levels=7, seed=99)
    ctx.device_status()
    covered = torch.zeros(w.M, dtype=torch.bool)
    for o, m in zip(w.layer_off, w.layer_len):
        covered[o:o + m] = True
    want = g_hat.cpu()
    assert torch.isfinite(out[covered]).all()
    # the chunks split tiles differently, which changes the fp32 order of the sum over nodes inside a tile only
    assert rel_l2(out[covered].numpy(), want[covered].numpy()) <= 1e-6
    with pytest.raises(gvq.GvqError):
        ctx.allreduce_host(g_pinned, Ut, mu, out, levels=128, seed=99)
