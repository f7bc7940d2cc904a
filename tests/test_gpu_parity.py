"""CUDA path vs the CPU oracle, element by element on the same seeded inputs, through the C ABI.

Tolerances (fp32 paths): relative L2 error <= 1e-5 on the compressed sum and on the
reconstructed gradient, per layer and over the whole buffer; bases compared through their
subspace (largest principal angle <= 1e-4 rad); quantizer levels and norms bit-exact.
"""
import numpy as np
import pytest
import torch

from paper_1811_03617_b200 import workloads as W
from util import layer_slices, rel_l2, subspace_angle

pytestmark = pytest.mark.gpu

TOL = 1e-5


@pytest.fixture(scope="module")
def gvq():
    from paper_1811_03617_b200 import gvq as _gvq
    _gvq.lib()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return _gvq


def _dev(x):
    return torch.as_tensor(np.ascontiguousarray(x)).cuda()


def _run_stream(gvq, w, g_dev, Ut_dev, mu_dev, per_node=False, path=0):
    ctx = gvq.Context(w)
    ctx.set_projection_path(path)
    s_sum = torch.full((ctx.S, w.k), float("nan"), device="cuda")
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    s_nodes = [torch.full((ctx.S, w.k), float("nan"), device="cuda") for _ in g_dev] if per_node else None
    ctx.compress_aggregate(g_dev, Ut_dev, mu_dev, s_sum, s_nodes)
    ctx.decompress(s_sum, Ut_dev, mu_dev, g_dev, len(g_dev), g_hat)
    ctx.device_status()  # waits for the stream; raises if a kernel gave up on a bounded wait
    return ctx, s_sum, g_hat, s_nodes


def _check_stream(w, oracle, g_np, Ut, mu, s_sum, g_hat, s_nodes=None):
    N = len(g_np)
    o_s_nodes = [oracle.compress(w, g, Ut, mu, N) for g in g_np]
    o_s = oracle.aggregate(o_s_nodes)
    o_g = oracle.decompress(w, o_s, Ut, mu, g_np, N, w.M)
    s_sum, g_hat = s_sum.cpu().numpy(), g_hat.cpu().numpy()
    covered = np.zeros(w.M, dtype=bool)
    for l in range(w.n_layers):
        (a, b), (sa, sb), (ta, tb) = layer_slices(w, l)
        covered[a:tb] = True
        if sb > sa:
            assert rel_l2(s_sum[sa:sb], o_s[sa:sb]) <= TOL, f"s_sum layer {l}"
            assert rel_l2(g_hat[a:b], o_g[a:b]) <= TOL, f"g_hat layer {l}"
        if tb > ta:
            # the tail is an fp32 sum in node order: bit-exact against that definition, and close to fp64
            seq = g_np[0][ta:tb].copy()
            for n in range(1, N):
                seq = seq + g_np[n][ta:tb]
            assert np.array_equal(g_hat[ta:tb], seq), f"tail layer {l}"
            assert np.allclose(g_hat[ta:tb], o_g[ta:tb], rtol=1e-5, atol=1e-5)
    assert rel_l2(s_sum, o_s) <= TOL
    assert rel_l2(g_hat[covered], o_g[covered]) <= TOL
    assert np.all(np.isnan(g_hat[~covered])), "entries outside every layer must not be written"
    if s_nodes is not None:
        for n in range(N):
            assert rel_l2(s_nodes[n].cpu().numpy(), o_s_nodes[n]) <= TOL, f"s_node {n}"
    return o_s, o_g


# ------------------------------------------------------------------------------ streaming path
@pytest.mark.parametrize("name", ["tiny", "resnet32"])
def test_stream_small_configs_with_fitted_basis(gvq, oracle, name):
    w = W.WORKLOADS[name]()
    hist = W.stored_gradients(w).numpy()
    Ut64, mu64, _, _ = oracle.fit_basis(w, hist, N=w.N, samples_are_sums_of=w.N)
    Ut, mu = Ut64.astype(np.float32), mu64.astype(np.float32)
    g = [t.numpy() for t in W.node_gradients(w, iteration=w.L)]
    ctx, s_sum, g_hat, s_nodes = _run_stream(gvq, w, [_dev(x) for x in g], _dev(Ut), _dev(mu), per_node=True)
    o_s, o_g = _check_stream(w, oracle, g, Ut, mu, s_sum, g_hat, s_nodes)
    # the data are rank k + small noise: the lossy aggregate is close to the true one
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    assert rel_l2(o_g, gsum) < 0.08


@pytest.mark.parametrize("path", [1, 2], ids=["fp32_pipe", "tensor_core"])
def test_stream_vgg16_shape(gvq, oracle, path):
    w = W.vgg16()
    Ut_t, mu_t = W.random_basis(w)
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx, s_sum, g_hat, _ = _run_stream(gvq, w, g_dev, Ut_t.cuda(), mu_t.cuda(), path=path)
    _check_stream(w, oracle, [x.cpu().numpy() for x in g_dev], Ut_t.numpy(), mu_t.numpy(), s_sum, g_hat)


def _gapped_offsets(lens):
    """Offsets that leave a gap between the layers: multiples of 4, but not of d."""
    off, acc = [], 8
    for m in lens:
        off.append(acc)
        acc += (m + 3) // 4 * 4 + 4
    return off


EDGE = [
    # name, d, k, N, layer_len                      what it covers
    ("ragged", 16, 4, 3, [16 * 257 + 5, 7, 16 * 255, 16, 16 * 1 + 15, 16 * 300]),   # tails, a layer < d, 1 slice
    ("full_rank16", 16, 16, 2, [16 * 100 + 4]),                                      # k = d
    ("full_rank64", 64, 64, 3, [64 * 70, 64 * 300 + 60]),                            # k = d, two passes
    ("k1", 32, 1, 4, [32 * 513]),                                                    # k = 1
    ("n1", 64, 8, 1, [64 * 40 + 8]),                                                 # N = 1
    ("n64", 16, 4, 64, [16 * 33]),                                                   # N at the limit
    ("d4", 4, 2, 2, [4 * 1000 + 3]),                                                 # smallest d
    ("d12k5", 12, 5, 3, [12 * 77 + 8]),                                              # d, k not powers of two
    ("d128k16", 128, 16, 5, [128 * 259, 128 * 3 + 100]),
    ("d256k32", 256, 32, 3, [256 * 130 + 192, 256 * 257]),
    ("d512k24", 512, 24, 2, [512 * 65 + 4]),
    ("d128k128", 128, 128, 2, [128 * 50]),                                           # widest k
]


TC_EDGE = [
    # shapes the tensor-core projection serves; slice counts around its 128-slice tile
    ("tc_d64k16", 64, 16, 3, [64 * 129 + 8, 64 * 1, 64 * 127, 64 * 128, 20, 64 * 300 + 60]),
    ("tc_d128k16", 128, 16, 5, [128 * 259, 128 * 3 + 100]),
    ("tc_d128k32", 128, 32, 2, [128 * 33 + 4]),
    ("tc_d192k32", 192, 32, 3, [192 * 140, 192 * 31]),
    ("tc_d256k32_n1", 256, 32, 1, [256 * 130 + 192]),
    ("tc_d256k32", 256, 32, 7, [256 * 130 + 192, 256 * 257, 256 * 5]),
    ("tc_d256k16_n64", 256, 16, 64, [256 * 40 + 12]),
]


@pytest.mark.parametrize("path", [1, 2], ids=["fp32_pipe", "tensor_core"])
@pytest.mark.parametrize("case", TC_EDGE, ids=[c[0] for c in TC_EDGE])
def test_stream_tensor_core_shapes(gvq, oracle, case, path):
    name, d, k, N, lens = case
    w = W.custom(name, 250 + len(name), d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    ctx, s_sum, g_hat, _ = _run_stream(gvq, w, [_dev(x) for x in g], Ut_t.cuda(), mu_t.cuda(), path=path)
    _check_stream(w, oracle, g, Ut_t.numpy(), mu_t.numpy(), s_sum, g_hat)
    # a single node through gvq_compress takes the same kernel
    s1 = torch.full((ctx.S, w.k), float("nan"), device="cuda")
    ctx.compress(_dev(g[0]), Ut_t.cuda(), mu_t.cuda(), w.N, s1)
    ctx.device_status()
    assert rel_l2(s1.cpu().numpy(), oracle.compress(w, g[0], Ut_t.numpy(), mu_t.numpy(), w.N)) <= TOL


@pytest.mark.parametrize("case", EDGE, ids=[c[0] for c in EDGE])
def test_stream_edge_cases(gvq, oracle, case):
    name, d, k, N, lens = case
    w = W.custom(name, 200 + len(name), d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    ctx, s_sum, g_hat, s_nodes = _run_stream(gvq, w, [_dev(x) for x in g], Ut_t.cuda(), mu_t.cuda(), per_node=True)
    _check_stream(w, oracle, g, Ut_t.numpy(), mu_t.numpy(), s_sum, g_hat, s_nodes)
    if k == d:  # lossless: the sum itself comes back
        gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
        for l in range(w.n_layers):
            (a, b), _, _ = layer_slices(w, l)
            if b > a:
                assert rel_l2(g_hat.cpu().numpy()[a:b], gsum[a:b]) <= 2e-5


def _random_layout(seed):
    """A seeded random layout: shape from the supported families, 1 - 9 layers of ragged lengths (empty layers,
    layers shorter than a slice, slice counts around the tile sizes), gaps between the layers."""
    rng = np.random.default_rng(1000 + seed)
    d, k = [(16, 4), (64, 8), (64, 16), (128, 16), (128, 32), (192, 32), (256, 16), (256, 32), (32, 32), (12, 5)][seed % 10]
    N = int(rng.integers(1, 9))
    lens = []
    for _ in range(int(rng.integers(1, 10))):
        kind = rng.integers(0, 6)
        if kind == 0:
            S = 0
        elif kind == 1:
            S = int(rng.choice([127, 128, 129, 255, 256, 257, 511, 512, 513, 64, 1]))
        else:
            S = int(rng.integers(1, 900))
        tail = int(rng.integers(0, d)) if rng.integers(0, 2) else 0
        lens.append(S * d + tail)
    if sum(m // d for m in lens) == 0:
        lens.append(d * 130 + 3)
    return W.custom(f"rand{seed}", 900 + seed, d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))


@pytest.mark.parametrize("seed", range(20))
def test_stream_random_layouts(gvq, oracle, seed):
    """Twenty seeded random layouts through the default path (and, where the shape has both, the other one):
    every entry against the oracle, per-node outputs included."""
    w = _random_layout(seed)
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [_dev(x) for x in g]
    ctx, s_sum, g_hat, s_nodes = _run_stream(gvq, w, g_dev, Ut_t.cuda(), mu_t.cuda(), per_node=True)
    _check_stream(w, oracle, g, Ut_t.numpy(), mu_t.numpy(), s_sum, g_hat, s_nodes)
    try:
        ctx.set_projection_path(2)
    except gvq.GvqError:
        return
    ctx2, s2, h2, _ = _run_stream(gvq, w, g_dev, Ut_t.cuda(), mu_t.cuda(), path=1)
    _check_stream(w, oracle, g, Ut_t.numpy(), mu_t.numpy(), s2, h2)


@pytest.mark.parametrize("d,k", [(16, 4), (128, 16)], ids=["fp32_pipe", "tensor_core_shape"])
def test_layout_without_any_full_slice(gvq, oracle, d, k):
    """The degenerate input: every layer shorter than a slice.  Nothing is compressed; the path is the plain sum of
    the tails, the compressed buffers are empty, the fit returns unit vectors."""
    lens = [d - 4, 8, d // 2]
    w = W.custom("all_tail", 12, d=d, k=k, N=3, L=2, layer_len=lens, layer_off=_gapped_offsets(lens))
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [_dev(x) for x in g]
    ctx = gvq.Context(w)
    assert ctx.S == 0
    Ut_t, mu_t = W.random_basis(w)
    s_sum = torch.zeros((1, k), device="cuda")      # a non-null pointer; no row of it is a slice
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    ctx.compress_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), s_sum)
    ctx.decompress(s_sum, Ut_t.cuda(), mu_t.cuda(), g_dev, w.N, g_hat)
    ctx.device_status()
    assert torch.all(s_sum == 0)
    got = g_hat.cpu().numpy()
    for l in range(w.n_layers):
        a, m = w.layer_off[l], w.layer_len[l]
        seq = g[0][a:a + m].copy()
        for n in range(1, w.N):
            seq = seq + g[n][a:a + m]
        assert np.array_equal(got[a:a + m], seq)
    o_g = oracle.decompress(w, np.zeros((0, k)), Ut_t.numpy(), mu_t.numpy(), g, w.N, w.M)
    cov = np.zeros(w.M, dtype=bool)
    for a, m in zip(w.layer_off, w.layer_len):
        cov[a:a + m] = True
    assert np.array_equal(np.isnan(got), ~cov) and np.allclose(got[cov], o_g[cov], rtol=1e-6, atol=1e-6)
    Ut = torch.full((w.n_layers, k, d), float("nan"), device="cuda")
    mu = torch.full((w.n_layers, d), float("nan"), device="cuda")
    ev = torch.full((w.n_layers, d), float("nan"), device="cuda")
    ctx.fit_basis(W.stored_gradients(w).cuda(), w.N, w.N, Ut, mu, ev)
    assert torch.equal(Ut.cpu(), torch.eye(d)[:k].expand(w.n_layers, k, d)) and torch.all(mu == 0) and torch.all(ev == 0)


def test_compress_then_aggregate_equals_fused(gvq, oracle):
    w = W.resnet32()
    Ut_t, mu_t = W.random_basis(w)
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx = gvq.Context(w)
    s_nodes = [torch.empty((ctx.S, w.k), device="cuda") for _ in range(w.N)]
    for n in range(w.N):
        ctx.compress(g_dev[n], Ut_t.cuda(), mu_t.cuda(), w.N, s_nodes[n])
    s_two_step = torch.empty((ctx.S, w.k), device="cuda")
    ctx.aggregate(s_nodes, s_two_step)
    s_fused = torch.empty((ctx.S, w.k), device="cuda")
    ctx.compress_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), s_fused)
    torch.cuda.synchronize()
    g_np = [x.cpu().numpy() for x in g_dev]
    for n in (0, w.N - 1):
        assert rel_l2(s_nodes[n].cpu().numpy(), oracle.compress(w, g_np[n], Ut_t.numpy(), mu_t.numpy(), w.N)) <= TOL
    o_s = oracle.aggregate([oracle.compress(w, g, Ut_t.numpy(), mu_t.numpy(), w.N) for g in g_np])
    assert rel_l2(s_two_step.cpu().numpy(), o_s) <= TOL
    assert rel_l2(s_fused.cpu().numpy(), o_s) <= TOL
    # Eq. 4: aggregate is the plain fp32 sum in node order -- bit-exact against that definition
    seq = s_nodes[0].cpu().numpy().copy()
    for n in range(1, w.N):
        seq = seq + s_nodes[n].cpu().numpy()
    assert np.array_equal(s_two_step.cpu().numpy(), seq)


def test_back_to_back_launches_stay_ordered_and_repeatable(gvq, oracle):
    """The two tensor-core kernels start their set-up while their predecessor in the stream still runs; what they
    read and write must stay ordered as in a plain stream.  A chain without host synchronisation: aggregate two
    groups of nodes, then aggregate the two reconstructions (the second projection reads what the decompression
    just wrote), twice over, bit-identical both times."""
    lens = [256 * 300 + 64, 256 * 129, 256 * 40]
    w = W.custom("chain", 303, d=256, k=32, N=4, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [_dev(x) for x in g]
    ctx = gvq.Context(w)
    outs = []
    for rep in range(2):
        s1 = torch.empty((ctx.S, w.k), device="cuda"); s2 = torch.empty_like(s1); s3 = torch.empty_like(s1)
        h1 = torch.zeros(w.M, device="cuda"); h2 = torch.zeros(w.M, device="cuda"); h3 = torch.zeros(w.M, device="cuda")
        ctx.compress_aggregate(g_dev[:2], Ut, mu, s1)
        ctx.decompress(s1, Ut, mu, g_dev[:2], 2, h1)
        ctx.compress_aggregate(g_dev[2:], Ut, mu, s2)
        ctx.decompress(s2, Ut, mu, g_dev[2:], 2, h2)
        ctx.compress_aggregate([h1, h2], Ut, mu, s3)          # reads the two buffers written just before
        ctx.decompress(s3, Ut, mu, [h1, h2], 2, h3)
        ctx.device_status()
        outs.append((s3.clone(), h3.clone()))
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    # against the oracle, step by step
    Utn, mun = Ut_t.numpy(), mu_t.numpy()
    def stage(nodes):
        o_s = oracle.aggregate([oracle.compress(w, x, Utn, mun, 2) for x in nodes])
        return oracle.decompress(w, o_s, Utn, mun, nodes, 2, w.M)
    o1, o2 = stage(g[:2]), stage(g[2:])
    o3 = stage([o1.astype(np.float32), o2.astype(np.float32)])
    covered = np.zeros(w.M, dtype=bool)
    for l in range(w.n_layers):
        covered[w.layer_off[l]:w.layer_off[l] + w.layer_len[l]] = True
    assert rel_l2(outs[0][1].cpu().numpy()[covered], o3[covered]) <= 3 * TOL


@pytest.mark.parametrize("name", ["resnet32", "tc_small"])
def test_step_can_be_captured_in_a_cuda_graph(gvq, name):
    """After one eager call (which caches the tensor maps of the buffers) the streaming calls only launch kernels,
    so a training loop may capture them in a CUDA graph; the replay gives the eager result bit for bit."""
    w = W.resnet32() if name == "resnet32" else W.custom("tc_small", 304, d=128, k=16, N=4, L=1,
                                                         layer_len=[128 * 300 + 40, 128 * 129])
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx = gvq.Context(w)
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    g_hat = torch.zeros(w.M, device="cuda")

    def step():
        ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
        ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()
    torch.cuda.synchronize()
    want = g_hat.clone()
    g_hat.zero_()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
        step()
    graph.replay()
    torch.cuda.synchronize()
    ctx.device_status()
    assert torch.equal(g_hat, want)


def test_allreduce_host_matches_device_path(gvq, oracle):
    w = W.custom("hostpath", 301, d=64, k=8, N=4, L=1, layer_len=[64 * 300 + 20, 64 * 129])
    Ut_t, mu_t = W.random_basis(w)
    g = W.node_gradients(w)
    ctx = gvq.Context(w)
    g_pinned = [x.pin_memory() for x in g]
    out = torch.empty(w.M, dtype=torch.float32).pin_memory()
    ctx.allreduce_host(g_pinned, Ut_t.cuda(), mu_t.cuda(), out)
    g_np = [x.numpy() for x in g]
    _, o_g = oracle.pipeline(w, g_np, Ut_t.numpy(), mu_t.numpy())
    assert rel_l2(out.numpy(), o_g) <= TOL


def test_allreduce_host_in_chunks_matches_device_path(gvq):
    """A gradient large enough for the host call to work through it in chunks (inputs of chunk c + 1 arriving while
    the result of chunk c leaves): same values as the device calls on the same inputs, tails and gaps included."""
    base = W.resnet50()
    w = W.custom("hostchunks", 302, d=base.d, k=base.k, N=3, L=1, layer_len=base.layer_len)
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g_dev = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx, s_sum, g_hat, _ = _run_stream(gvq, w, g_dev, Ut, mu)
    g_pinned = [x.cpu().pin_memory() for x in g_dev]
    out = torch.full((w.M,), float("nan")).pin_memory()
    ctx.ensure_workspace(ctx.layout.host_workspace_bytes(w.N))
    ctx.host_prepare()           # builds the chunk contexts (the call itself allocates nothing)
    for _ in range(2):           # the second call reuses the chunk contexts and their tensor maps
        out.fill_(float("nan"))
        ctx.allreduce_host(g_pinned, Ut, mu, out)
        ctx.device_status()
        want = g_hat.cpu()
        covered = torch.zeros(w.M, dtype=torch.bool)
        for o, m in zip(w.layer_off, w.layer_len):
            covered[o:o + m] = True
        assert torch.isfinite(out[covered]).all()
        assert rel_l2(out[covered].numpy(), want[covered].numpy()) <= 1e-6
        for l in range(w.n_layers):    # the tails are fp32 sums in node order on both routes
            _, _, (ta, tb) = layer_slices(w, l)
            assert torch.equal(out[ta:tb], want[ta:tb])


# ------------------------------------------------------------------------------ full-size, sampled
def _sampled_check(gvq, oracle, w, n_samples, seed, path=0):
    """Runs the path at full size on device-generated inputs and checks sampled slices one by one."""
    Ut_t, mu_t = W.random_basis(w)
    g_dev = [W.node_gradient(w, n, iteration=w.L, device="cuda") for n in range(w.N)]
    ctx, s_sum, g_hat, _ = _run_stream(gvq, w, g_dev, Ut_t.cuda(), mu_t.cuda(), path=path)
    rng = np.random.default_rng(seed)
    Ut, mu = Ut_t.numpy(), mu_t.numpy()
    worst_s = worst_g = 0.0
    # per layer: first, last and a few random slices (the last tile of a layer is ragged)
    for l in range(w.n_layers):
        S = w.layer_len[l] // w.d
        if S == 0:
            continue
        (a, b), (sa, sb), (ta, tb) = layer_slices(w, l)
        rows = np.unique(np.concatenate([[0, S - 1, min(S - 1, 255), min(S - 1, 256)],
                                         rng.integers(0, S, n_samples)]))
        idx = torch.as_tensor((a + rows[:, None] * w.d + np.arange(w.d)[None, :]).ravel(), device="cuda")
        xs = [g[idx].cpu().numpy().reshape(len(rows), w.d) for g in g_dev]
        mini = W.custom("mini", 1, d=w.d, k=w.k, N=w.N, L=1, layer_len=[len(rows) * w.d])
        o_s, o_g = oracle.pipeline(mini, [x.ravel() for x in xs], Ut[l:l + 1], mu[l:l + 1])
        got_s = s_sum[torch.as_tensor(sa + rows, device="cuda")].cpu().numpy()
        got_g = g_hat[idx].cpu().numpy()
        worst_s = max(worst_s, rel_l2(got_s, o_s))
        worst_g = max(worst_g, rel_l2(got_g, o_g))
        if tb > ta:
            seq = g_dev[0][ta:tb].clone()
            for n in range(1, w.N):
                seq += g_dev[n][ta:tb]
            assert torch.equal(g_hat[ta:tb], seq)
    assert worst_s <= TOL and worst_g <= TOL, (worst_s, worst_g)
    assert torch.isfinite(s_sum).all() and torch.isfinite(g_hat).all()
    return ctx, g_dev, s_sum, g_hat


@pytest.mark.parametrize("path", [1, 0], ids=["fp32_pipe", "default"])
def test_stream_resnet50_full_size_every_element(gvq, oracle, path):
    """The ResNet-50-shaped configuration at full size, every entry of s_sum and g_hat against the oracle."""
    w = W.resnet50()
    Ut_t, mu_t = W.random_basis(w)
    g_dev = [W.node_gradient(w, n, iteration=w.L, device="cuda") for n in range(w.N)]
    ctx, s_sum, g_hat, _ = _run_stream(gvq, w, g_dev, Ut_t.cuda(), mu_t.cuda(), path=path)
    _check_stream(w, oracle, [x.cpu().numpy() for x in g_dev], Ut_t.numpy(), mu_t.numpy(), s_sum, g_hat)


def _whole_layers(w, layers):
    """A layout of its own made of the given layers of w, packed; plus the index ranges that map it back."""
    sub = W.custom(w.name + "_layers", 1, d=w.d, k=w.k, N=w.N, L=w.L, layer_len=[w.layer_len[l] for l in layers])
    flat = torch.cat([torch.arange(w.layer_off[l], w.layer_off[l] + w.layer_len[l]) for l in layers])
    rows = torch.cat([torch.arange(layer_slices(w, l)[1][0], layer_slices(w, l)[1][1]) for l in layers])
    return sub, flat, rows


LARGE_WHOLE_LAYERS = (0, 1, 30, 57, 58)   # first (1x1), a 3x3, a middle 1x1, the last 3x3, last (1x1)


def test_stream_large_full_size(gvq, oracle):
    """The 100 M-entry configuration at full size without its quantizer: every slice of five whole layers against the
    oracle, sampled slices of all the others."""
    free, _ = torch.cuda.mem_get_info()
    w = W.large()
    if free < (w.N + 2) * w.M * 4 + (2 << 30):
        pytest.skip("not enough free device memory for the 100M-entry workload")
    ctx, g_dev, s_sum, g_hat = _sampled_check(gvq, oracle, w, 12, 5)
    sub, flat, rows = _whole_layers(w, LARGE_WHOLE_LAYERS)
    flat_d, rows_d = flat.cuda(), rows.cuda()
    Ut_t, mu_t = W.random_basis(w)
    idx = list(LARGE_WHOLE_LAYERS)
    o_s, o_g = oracle.pipeline(sub, [g[flat_d].cpu().numpy() for g in g_dev], Ut_t.numpy()[idx], mu_t.numpy()[idx])
    got_s, got_g = s_sum[rows_d].cpu().numpy(), g_hat[flat_d].cpu().numpy()
    for j in range(len(idx)):
        (a, b), (sa, sb), _ = layer_slices(sub, j)
        assert rel_l2(got_s[sa:sb], o_s[sa:sb]) <= TOL and rel_l2(got_g[a:b], o_g[a:b]) <= TOL, f"layer {idx[j]}"


# ------------------------------------------------------------------------------ quantizer
# ------------------------------------------------------------------------------ Eq. 7 monitor
MON = [
    # name, d, k, N, layer_len, tensor-core shape?
    ("mon_tc_d128k16", 128, 16, 5, [128 * 259, 128 * 3 + 100, 40, 128 * 128], True),
    ("mon_tc_d256k32", 256, 32, 7, [256 * 130 + 192, 256 * 257, 256 * 5], True),
    ("mon_tc_d64k16_n64", 64, 16, 64, [64 * 300 + 12, 64 * 1], True),
    ("mon_fp32_d64k8", 64, 8, 4, [64 * 300 + 20, 64 * 129, 30], False),
    ("mon_fp32_d12k5", 12, 5, 3, [12 * 77 + 8], False),
]


def _single_layer(w, l):
    return W.custom(w.name + f"_l{l}", 1, d=w.d, k=w.k, N=w.N, L=1, layer_len=[w.layer_len[l]], layer_off=[0])


@pytest.mark.parametrize("case", MON, ids=[c[0] for c in MON])
def test_local_loss_monitor(gvq, oracle, case):
    """Eq. 7 per layer and node: energy against its definition, energy - captured against the oracle's literal
    residual.  The loss is a difference of two fp32-accumulated sums and the random basis is orthonormal to fp32
    rounding, so the bar is absolute: 3e-5 of the energy."""
    name, d, k, N, lens, tc = case
    w = W.custom(name, 400 + len(name), d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [_dev(x) for x in g]
    ctx = gvq.Context(w)
    s_ref = torch.empty((ctx.S, w.k), device="cuda")
    ctx.compress_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), s_ref)
    s_sum = torch.full((ctx.S, w.k), float("nan"), device="cuda")
    mon = torch.full((w.n_layers, 2, N), float("nan"), dtype=torch.float64, device="cuda")
    s_nodes = None if tc else [torch.empty((ctx.S, w.k), device="cuda") for _ in range(N)]
    if not tc:
        with pytest.raises(gvq.GvqError):   # no fused form for this shape: the per-node outputs are required
            ctx.compress_aggregate_monitored(g_dev, Ut_t.cuda(), mu_t.cuda(), s_sum, mon)
    for _ in range(2):   # the second call must overwrite, not accumulate
        ctx.compress_aggregate_monitored(g_dev, Ut_t.cuda(), mu_t.cuda(), s_sum, mon, s_nodes)
    ctx.device_status()
    if tc:
        assert torch.equal(s_sum, s_ref), "the monitor must not change the compressed sum"
    else:
        assert rel_l2(s_sum.cpu().numpy(), s_ref.cpu().numpy()) <= 1e-6
    mon = mon.cpu().numpy()
    Ut, mu = Ut_t.numpy(), mu_t.numpy()
    for l in range(w.n_layers):
        (a, b), _, _ = layer_slices(w, l)
        wl = _single_layer(w, l)
        for n in range(N):
            if b == a:
                assert mon[l, 0, n] == 0.0 and mon[l, 1, n] == 0.0
                continue
            xc = g[n][a:b].astype(np.float64).reshape(-1, d) - mu[l].astype(np.float64) / N
            energy = float((xc ** 2).sum())
            assert abs(mon[l, 0, n] - energy) <= 2e-6 * energy, (l, n)
            loss = oracle.local_loss(wl, g[n][w.layer_off[l]:w.layer_off[l] + w.layer_len[l]], Ut[l:l + 1], mu[l:l + 1], N)
            assert abs((mon[l, 0, n] - mon[l, 1, n]) - loss) <= 3e-5 * energy, (l, n, loss, energy)
            assert 0.0 <= loss <= energy * (1 + 1e-12)


def test_local_loss_monitor_sees_a_stale_basis(gvq, oracle):
    """The use the paper makes of Eq. 7: with the fitted basis the relative loss is the noise floor; after the
    gradients' subspace has moved it is large on every node."""
    w = W.custom("mon_drift", 77, d=128, k=16, N=4, L=4, layer_len=[128 * 600, 128 * 300 + 64])
    hist = W.stored_gradients(w, device="cuda")
    ctx = gvq.Context(w)
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda"); mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    ctx.fit_basis(hist, w.N, w.N, Ut, mu, ev)
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    mon = torch.empty((w.n_layers, 2, w.N), dtype=torch.float64, device="cuda")
    g_dev = [W.node_gradient(w, n, iteration=w.L, device="cuda") for n in range(w.N)]
    ctx.compress_aggregate_monitored(g_dev, Ut, mu, s_sum, mon)
    fresh = (1.0 - mon[:, 1] / mon[:, 0]).cpu().numpy()
    # a basis of another subspace: the rows of Ut rolled along the slice
    ctx.compress_aggregate_monitored(g_dev, torch.roll(Ut, 7, dims=2).contiguous(), mu, s_sum, mon)
    stale = (1.0 - mon[:, 1] / mon[:, 0]).cpu().numpy()
    assert np.all(fresh < 0.02) and np.all(stale > 0.5), (fresh, stale)



@pytest.mark.parametrize("path", [1, 2], ids=["fp32_pipe", "tensor_core"])
def test_per_layer_k_through_a_masked_basis(gvq, oracle, path):
    """Eq. 6 picks a k_l per layer; with rows k_l.. of a layer's basis zeroed the k-wide buffers carry exact zeros
    there and the path computes what the oracle computes with k_l columns."""
    lens = [128 * 259, 128 * 3 + 100, 128 * 140, 128 * 64]
    w = W.custom("perlayer_k", 91, d=128, k=16, N=3, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    ks = [16, 5, 0, 9]
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [_dev(x) for x in g]
    ctx = gvq.Context(w)
    ctx.set_projection_path(path)
    Ut_dev = Ut_t.cuda()
    ctx.mask_basis(Ut_dev, ks)
    with pytest.raises(gvq.GvqError):
        ctx.mask_basis(Ut_dev, [17, 0, 0, 0])
    s_sum = torch.full((ctx.S, w.k), float("nan"), device="cuda")
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    ctx.compress_aggregate(g_dev, Ut_dev, mu_t.cuda(), s_sum)
    ctx.decompress(s_sum, Ut_dev, mu_t.cuda(), g_dev, w.N, g_hat)
    ctx.device_status()
    s_sum, g_hat = s_sum.cpu().numpy(), g_hat.cpu().numpy()
    Ut, mu = Ut_t.numpy(), mu_t.numpy()
    for l, kl in enumerate(ks):
        (a, b), (sa, sb), _ = layer_slices(w, l)
        assert np.all(s_sum[sa:sb, kl:] == 0.0), "masked coordinates are exact zeros"
        seg = [x[w.layer_off[l]:w.layer_off[l] + w.layer_len[l]] for x in g]
        if kl == 0:   # nothing is kept: the reconstruction is the mean
            assert np.allclose(g_hat[a:b].reshape(-1, w.d), mu[l][None, :], rtol=0, atol=1e-6)
            continue
        wl = W.custom(f"perlayer_k_l{l}", 1, d=w.d, k=kl, N=w.N, L=1, layer_len=[lens[l]], layer_off=[0])
        Ul, ml = np.ascontiguousarray(Ut[l:l + 1, :kl]), mu[l:l + 1]
        o_s = oracle.aggregate([oracle.compress(wl, x, Ul, ml, w.N) for x in seg])
        o_g = oracle.decompress(wl, o_s, Ul, ml, seg, w.N, lens[l])
        assert rel_l2(s_sum[sa:sb, :kl], o_s) <= TOL
        assert rel_l2(g_hat[a:b], o_g[:b - a]) <= TOL


@pytest.mark.parametrize("k,levels", [(4, 7), (8, 1), (16, 127), (32, 7), (5, 7), (1, 3)])
def test_quantize_bit_exact(gvq, oracle, k, levels):
    d = 32 if k <= 32 else 64
    w = W.custom("q", 400 + k, d=d, k=k, N=3, L=1, layer_len=[d * 1000 + 4, d * 531])
    ctx = gvq.Context(w)
    rng = np.random.default_rng(k * 131 + levels)
    qs, ns, o_qs, o_ns, s_list = [], [], [], [], []
    for node in range(w.N):
        s = rng.standard_normal((ctx.S, k)).astype(np.float32) * np.float32(10.0 ** rng.integers(-3, 4))
        s_list.append(s)
        s[5] = 0.0
        s[6, 1:] = 0.0
        s[7] = np.float32(-0.0)
        q = torch.full((ctx.S, k), 99, dtype=torch.int8, device="cuda")
        norms = torch.full((ctx.S,), float("nan"), device="cuda")
        ctx.quantize(_dev(s), levels, 20181103, node, q, norms)
        o_q, o_n = oracle.quantize(s, levels, 20181103, node)
        assert np.array_equal(q.cpu().numpy(), o_q)
        assert np.array_equal(norms.cpu().numpy(), o_n)
        qs.append(q); ns.append(norms); o_qs.append(o_q); o_ns.append(o_n)
    out = torch.empty((ctx.S, k), device="cuda")
    ctx.dequantize_aggregate(qs, ns, levels, out)
    assert rel_l2(out.cpu().numpy(), oracle.dequantize_aggregate(o_qs, o_ns, levels)) <= 1e-6
    # the single-launch form over all nodes is bit-identical to the separate calls
    s_in = [_dev(x) for x in s_list]
    q2 = [torch.full((ctx.S, k), 99, dtype=torch.int8, device="cuda") for _ in range(w.N)]
    n2 = [torch.full((ctx.S,), float("nan"), device="cuda") for _ in range(w.N)]
    out2 = torch.full((ctx.S, k), float("nan"), device="cuda")
    ctx.quantize_aggregate(s_in, levels, 20181103, out2, q2, n2)
    assert torch.equal(out2, out)
    assert all(torch.equal(a, b) for a, b in zip(q2, qs)) and all(torch.equal(a, b) for a, b in zip(n2, ns))
    out3 = torch.empty((ctx.S, k), device="cuda")
    ctx.quantize_aggregate(s_in, levels, 20181103, out3)
    assert torch.equal(out3, out)


def test_quantized_pipeline_end_to_end(gvq, oracle):
    """compress -> quantize each node -> dequantise-and-sum -> decompress, against the oracle."""
    w = W.custom("qpipe", 410, d=64, k=8, N=4, L=1, layer_len=[64 * 700 + 12, 64 * 259])
    levels, seed = 7, 77
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    ctx = gvq.Context(w)
    g_dev = [_dev(x) for x in g]
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    s_nodes = [torch.empty((ctx.S, w.k), device="cuda") for _ in g]
    ctx.compress_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), s_sum, s_nodes)
    qs = [torch.empty((ctx.S, w.k), dtype=torch.int8, device="cuda") for _ in g]
    ns = [torch.empty((ctx.S,), device="cuda") for _ in g]
    for n in range(w.N):
        ctx.quantize(s_nodes[n], levels, seed, n, qs[n], ns[n])
    sq = torch.empty((ctx.S, w.k), device="cuda")
    ctx.dequantize_aggregate(qs, ns, levels, sq)
    g_hat = torch.empty(w.M, device="cuda")
    ctx.decompress(sq, Ut_t.cuda(), mu_t.cuda(), g_dev, w.N, g_hat)
    torch.cuda.synchronize()
    Ut, mu = Ut_t.numpy(), mu_t.numpy()
    mism = total = 0
    flip2 = 0.0
    o_qs, o_ns = [], []
    for n in range(w.N):
        # (ii) the library's levels are bit-exact for the s_n it produced itself
        dumped = s_nodes[n].cpu().numpy()
        q_self, n_self = oracle.quantize(dumped, levels, seed, n)
        assert np.array_equal(qs[n].cpu().numpy(), q_self) and np.array_equal(ns[n].cpu().numpy(), n_self)
        # (iii) against the oracle's own s_n (fp64 -> fp32): only boundary cases may differ, by one level
        o_q, o_n = oracle.quantize(oracle.compress(w, g[n], Ut, mu, w.N).astype(np.float32), levels, seed, n)
        m, e2 = _flip_energy(qs[n].cpu().numpy(), o_q, o_n, levels)
        mism += m; total += o_q.size; flip2 += e2
        o_qs.append(o_q); o_ns.append(o_n)
    assert mism <= 1e-3 * total
    o_sq = oracle.dequantize_aggregate(o_qs, o_ns, levels)
    o_g = oracle.decompress(w, o_sq, Ut, mu, g, w.N, w.M)
    # a level flip moves one coordinate by norm / levels: allow for what the counted flips can move
    moved = 1.01 * np.sqrt(flip2)
    assert rel_l2(sq.cpu().numpy(), o_sq) <= 1e-5 + moved / np.linalg.norm(o_sq)
    assert rel_l2(g_hat.cpu().numpy(), o_g) <= 1e-5 + moved / np.linalg.norm(o_g)


def _flip_energy(got_q, o_q, o_n, levels):
    """What level flips can move: a flipped coordinate of a node's vector moves by norm / levels.  Returns
    (flipped coordinates, sum over them of (norm / levels)^2); asserts that no level differs by more than one."""
    diff = np.abs(got_q.astype(np.int32) - o_q.astype(np.int32))
    assert diff.max() <= 1
    step2 = (o_n.astype(np.float64) / levels) ** 2
    return int((diff != 0).sum()), float((diff != 0).sum(axis=1) @ step2)


QF = [("qf_d256k32", 256, 32, 5, [256 * 130 + 192, 256 * 257, 256 * 5]), ("qf_d128k16", 128, 16, 16, [128 * 300, 128 * 77 + 4]),
      ("qf_d64k16_n1", 64, 16, 1, [64 * 129])]


@pytest.mark.parametrize("case", QF, ids=[c[0] for c in QF])
def test_fused_compress_quantize_aggregate(gvq, oracle, case):
    """The one-pass form against the three separate calls and against the oracle."""
    name, d, k, N, lens = case
    levels, seed = 7, 4242
    w = W.custom(name, 430 + d, d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [_dev(x) for x in g]
    ctx = gvq.Context(w)
    S = ctx.S
    # separate calls: per-node s_n, quantize each, dequantise-and-sum
    s_tmp = torch.empty((S, k), device="cuda")
    s_nodes = [torch.empty((S, k), device="cuda") for _ in g]
    ctx.compress_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), s_tmp, s_nodes)
    qs = [torch.empty((S, k), dtype=torch.int8, device="cuda") for _ in g]
    ns = [torch.empty((S,), device="cuda") for _ in g]
    for n in range(N):
        ctx.quantize(s_nodes[n], levels, seed, n, qs[n], ns[n])
    s_sep = torch.empty((S, k), device="cuda")
    ctx.dequantize_aggregate(qs, ns, levels, s_sep)
    # one pass
    qf = [torch.full((S, k), 99, dtype=torch.int8, device="cuda") for _ in g]
    nf = [torch.full((S,), float("nan"), device="cuda") for _ in g]
    s_fused = torch.full((S, k), float("nan"), device="cuda")
    ctx.compress_quantize_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), levels, seed, s_fused, qf, nf)
    ctx.device_status()
    for n in range(N):
        assert torch.equal(qf[n], qs[n]), f"levels of node {n}"
        assert torch.equal(nf[n], ns[n]), f"norms of node {n}"
        # and both are bit-exact with the oracle's quantizer on the s_n the library produced
        o_q, o_n = oracle.quantize(s_nodes[n].cpu().numpy(), levels, seed, n)
        assert np.array_equal(qf[n].cpu().numpy(), o_q) and np.array_equal(nf[n].cpu().numpy(), o_n)
    assert rel_l2(s_fused.cpu().numpy(), s_sep.cpu().numpy()) <= 1e-6
    # without the optional outputs the sum is the same
    s2 = torch.empty((S, k), device="cuda")
    ctx.compress_quantize_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), levels, seed, s2)
    ctx.device_status()
    assert torch.equal(s2, s_fused)
    # end to end against the oracle: level flips only on decision boundaries
    Ut, mu = Ut_t.numpy(), mu_t.numpy()
    o_qs, o_ns, mism, total, flip2 = [], [], 0, 0, 0.0
    for n in range(N):
        o_q, o_n = oracle.quantize(oracle.compress(w, g[n], Ut, mu, N).astype(np.float32), levels, seed, n)
        m, e2 = _flip_energy(qf[n].cpu().numpy(), o_q, o_n, levels)
        mism += m; total += o_q.size; flip2 += e2
        o_qs.append(o_q); o_ns.append(o_n)
    assert mism <= 1e-3 * total
    o_sq = oracle.dequantize_aggregate(o_qs, o_ns, levels)
    assert rel_l2(s_fused.cpu().numpy(), o_sq) <= 1e-5 + 1.01 * np.sqrt(flip2) / np.linalg.norm(o_sq)


@pytest.mark.parametrize("seed", range(6))
def test_fused_quantize_random_layouts(gvq, oracle, seed):
    """Seeded random tensor-core layouts, levels and seeds through the one-pass call: what every node would transmit is
    bit-exact against the oracle's quantizer on the s_n the library dumps; the sum equals the separate calls'."""
    rng = np.random.default_rng(3000 + seed)
    d, k = [(64, 16), (128, 16), (128, 32), (192, 32), (256, 16), (256, 32)][seed]
    N, levels, qseed = int(rng.integers(1, 10)), int(rng.choice([1, 3, 7, 15, 127])), int(rng.integers(0, 2 ** 62))
    lens = [int(rng.choice([1, 127, 128, 129, 300, 513])) * d + (int(rng.integers(0, d)) if rng.integers(0, 2) else 0)
            for _ in range(int(rng.integers(1, 6)))]
    w = W.custom(f"randq{seed}", 970 + seed, d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    Ut_t, mu_t = W.random_basis(w)
    g_dev = [_dev(t.numpy()) for t in W.node_gradients(w)]
    ctx = gvq.Context(w)
    S = ctx.S
    s_tmp = torch.empty((S, k), device="cuda")
    s_nodes = [torch.empty((S, k), device="cuda") for _ in g_dev]
    ctx.compress_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), s_tmp, s_nodes)
    s_sep = torch.empty((S, k), device="cuda")
    ctx.quantize_aggregate(s_nodes, levels, qseed, s_sep)
    qf = [torch.full((S, k), 99, dtype=torch.int8, device="cuda") for _ in g_dev]
    nf = [torch.full((S,), float("nan"), device="cuda") for _ in g_dev]
    s_fused = torch.full((S, k), float("nan"), device="cuda")
    ctx.compress_quantize_aggregate(g_dev, Ut_t.cuda(), mu_t.cuda(), levels, qseed, s_fused, qf, nf)
    ctx.device_status()
    for n in range(N):
        o_q, o_n = oracle.quantize(s_nodes[n].cpu().numpy(), levels, qseed, n)
        assert np.array_equal(qf[n].cpu().numpy(), o_q) and np.array_equal(nf[n].cpu().numpy(), o_n), n
    assert rel_l2(s_fused.cpu().numpy(), s_sep.cpu().numpy()) <= 1e-6


def test_large_config_with_its_quantizer_at_full_size(gvq, oracle):
    """The largest configuration as specified -- 100 M entries, 32 nodes, 16-code quantizer on s -- through the
    one-pass call at full size.  (i) on whole layers the levels and norms are bit-exact against the oracle's
    quantizer applied to the s_n the library dumps (three-launch form, same inputs); (ii) the one-pass call's
    levels and norms equal the three-launch form's on every slice of every node; (iii) against the oracle end to
    end levels differ on decision boundaries only (<= 1e-3 of them, by one level) and s_sum / g_hat stay within the
    bound that implies."""
    w = W.large()
    free, _ = torch.cuda.mem_get_info()
    if free < (w.N + 2) * w.M * 4 + (6 << 30):
        pytest.skip("not enough free device memory for the 100M-entry workload with per-node outputs")
    levels, seed = 7, 20181103
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g_dev = [W.node_gradient(w, n, iteration=w.L, device="cuda") for n in range(w.N)]
    ctx = gvq.Context(w)
    S, k, N = ctx.S, w.k, w.N
    s_tmp = torch.empty((S, k), device="cuda")
    s_nodes = [torch.empty((S, k), device="cuda") for _ in range(N)]
    ctx.compress_aggregate(g_dev, Ut, mu, s_tmp, s_nodes)
    qs = [torch.full((S, k), 99, dtype=torch.int8, device="cuda") for _ in range(N)]
    ns = [torch.full((S,), float("nan"), device="cuda") for _ in range(N)]
    s_sep = torch.empty((S, k), device="cuda")
    ctx.quantize_aggregate(s_nodes, levels, seed, s_sep, qs, ns)
    qf = [torch.full((S, k), 99, dtype=torch.int8, device="cuda") for _ in range(N)]
    nf = [torch.full((S,), float("nan"), device="cuda") for _ in range(N)]
    s_fused = torch.full((S, k), float("nan"), device="cuda")
    ctx.compress_quantize_aggregate(g_dev, Ut, mu, levels, seed, s_fused, qf, nf)
    g_hat = torch.empty(w.M, device="cuda")
    ctx.decompress(s_fused, Ut, mu, g_dev, N, g_hat)
    ctx.device_status()
    for n in range(N):                                                        # (ii), full size
        assert torch.equal(qf[n], qs[n]), f"levels of node {n}"
        assert torch.equal(nf[n], ns[n]), f"norms of node {n}"
    assert rel_l2(s_fused.cpu().numpy(), s_sep.cpu().numpy()) <= 1e-6
    assert torch.isfinite(g_hat).all()
    sub, flat, rows = _whole_layers(w, LARGE_WHOLE_LAYERS)
    flat_d, rows_d = flat.cuda(), rows.cuda()
    idx = list(LARGE_WHOLE_LAYERS)
    Ut_s, mu_s = Ut_t.numpy()[idx], mu_t.numpy()[idx]
    g_sub = [g[flat_d].cpu().numpy() for g in g_dev]
    row0 = [layer_slices(w, l)[1][0] for l in idx]                            # a layer's first row in the whole layout
    o_qs, o_ns, mism, total, flip2 = [], [], 0, 0, 0.0
    for n in range(N):
        dumped = s_nodes[n][rows_d].cpu().numpy()
        got_q, got_n = qf[n][rows_d].cpu().numpy(), nf[n][rows_d].cpu().numpy()
        o_sn = oracle.compress(sub, g_sub[n], Ut_s, mu_s, N).astype(np.float32)
        oq_n, on_n = [], []
        for j in range(len(idx)):
            _, (sa, sb), _ = layer_slices(sub, j)
            q_self, n_self = oracle.quantize(dumped[sa:sb], levels, seed, n, slice0=row0[j])      # (i)
            assert np.array_equal(got_q[sa:sb], q_self) and np.array_equal(got_n[sa:sb], n_self), (n, idx[j])
            o_q, o_n = oracle.quantize(o_sn[sa:sb], levels, seed, n, slice0=row0[j])              # (iii)
            oq_n.append(o_q); on_n.append(o_n)
        o_q, o_n = np.concatenate(oq_n), np.concatenate(on_n)
        m, e2 = _flip_energy(got_q, o_q, o_n, levels)
        mism += m; total += o_q.size; flip2 += e2
        o_qs.append(o_q); o_ns.append(o_n)
    assert mism <= 1e-3 * total
    o_sq = oracle.dequantize_aggregate(o_qs, o_ns, levels)
    o_g = oracle.decompress(sub, o_sq, Ut_s, mu_s, g_sub, N, sub.M)
    # what the counted flips can move (Eq. 5 with orthonormal rows of Ut carries the same norm over to g_hat)
    moved = 1.01 * np.sqrt(flip2)
    assert rel_l2(s_fused[rows_d].cpu().numpy(), o_sq) <= 1e-5 + moved / np.linalg.norm(o_sq)
    assert rel_l2(g_hat[flat_d].cpu().numpy(), o_g) <= 1e-5 + moved / np.linalg.norm(o_g)


def test_fused_quantize_unsupported_shape(gvq):
    w = W.tiny()
    ctx = gvq.Context(w)
    Ut_t, mu_t = W.random_basis(w)
    g = [torch.zeros(w.M, device="cuda") for _ in range(w.N)]
    with pytest.raises(gvq.GvqError) as e:
        ctx.compress_quantize_aggregate(g, Ut_t.cuda(), mu_t.cuda(), 7, 1, torch.empty((ctx.S, w.k), device="cuda"))
    assert e.value.status == 4


# ------------------------------------------------------------------------------ basis fit
def _check_fit(w, oracle, hist_np, Ut_g, mu_g, ev_g, N, c, layers=None, tail_tol=1e-5):
    """Every eigenvalue within tail_tol = 1e-5 of the largest (absolute), on every fit path; their sum equal to the
    trace of the covariance to 1e-5 (Eq. 6 divides by it)."""
    o_Ut, o_mu, o_ev, _ = oracle.fit_basis(w, hist_np, N=N, samples_are_sums_of=c)
    worst = 0.0
    for l in (range(w.n_layers) if layers is None else layers):
        S = w.layer_len[l] // w.d
        G = Ut_g[l].astype(np.float64)
        assert np.abs(G @ G.T - np.eye(w.k)).max() <= 1e-5, f"orthonormality layer {l}"
        lam_max = max(o_ev[l, 0], 1e-30)
        assert np.abs(ev_g[l, : w.k] - o_ev[l, : w.k]).max() <= 1e-5 * lam_max, f"leading eigenvalues layer {l}"
        assert np.abs(ev_g[l] - o_ev[l]).max() <= tail_tol * lam_max, f"eigenvalues layer {l}"
        assert abs(ev_g[l].astype(np.float64).sum() - o_ev[l].sum()) <= 1e-5 * max(o_ev[l].sum(), 1e-30), f"trace layer {l}"
        assert np.all(np.diff(ev_g[l]) <= 0), "eigenvalues must be sorted descending"
        assert np.allclose(mu_g[l], o_mu[l], rtol=1e-5, atol=1e-6 * (np.abs(o_mu[l]).max() + 1e-30))
        if S == 0:
            assert np.array_equal(Ut_g[l], np.eye(w.d, dtype=np.float32)[: w.k])
            continue
        n = hist_np.shape[0] * S
        if n > w.k and o_ev[l, w.k - 1] > 10 * o_ev[l, min(w.k, w.d - 1)] and w.k < w.d:
            assert np.allclose(ev_g[l, : w.k], o_ev[l, : w.k], rtol=1e-4)
            ang = subspace_angle(G, o_Ut[l])
            worst = max(worst, ang)
            assert ang <= 1e-4, f"subspace angle layer {l}: {ang}"
            # sign convention: the largest-magnitude entry of every basis vector is positive
            big = np.abs(G).argmax(axis=1)
            assert np.all(G[np.arange(w.k), big] > 0)
    return worst


FIT_PATHS = pytest.mark.parametrize("fit_path", [1, 2], ids=["rotations_kept", "values_and_subspace"])
# bar on the eigenvalues after the k leading ones, in units of the largest, per fit path (0 = automatic = 2 here)
FIT_TAIL_TOL = {0: 1e-5, 1: 1e-5, 2: 1e-5}


@FIT_PATHS
@pytest.mark.parametrize("name", ["tiny", "resnet32"])
def test_fit_basis_small_configs(gvq, oracle, name, fit_path):
    w = W.WORKLOADS[name]()
    hist = W.stored_gradients(w)
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut = torch.full((w.n_layers, w.k, w.d), float("nan"), device="cuda")
    mu = torch.full((w.n_layers, w.d), float("nan"), device="cuda")
    ev = torch.full((w.n_layers, w.d), float("nan"), device="cuda")
    sweeps = ctx.fit_basis(hist.cuda(), w.N, w.N, Ut, mu, ev)
    assert all(0 < s < 30 for s in sweeps)
    _check_fit(w, oracle, hist.numpy(), Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), w.N, w.N,
               tail_tol=FIT_TAIL_TOL[fit_path])
    # the fitted basis does its job: compress/decompress of a fresh iteration loses little
    g = W.node_gradients(w, iteration=w.L)
    g_dev = [x.cuda() for x in g]
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    g_hat = torch.empty(w.M, device="cuda")
    ctx.compress_aggregate(g_dev, Ut, mu, s_sum)
    ctx.decompress(s_sum, Ut, mu, g_dev, w.N, g_hat)
    gsum = torch.stack(g_dev).double().sum(0)
    loss = float(((g_hat.double() - gsum) ** 2).sum() / (gsum ** 2).sum())
    assert loss < 0.01  # the paper's loss threshold lambda = 0.01


FIT_EDGE = [
    ("fit_d128", 128, 16, 4, 4, [128 * 300 + 17, 128 * 40, 60]),      # a layer without a full slice
    ("fit_d256", 256, 32, 2, 3, [256 * 200, 256 * 600 + 8]),
    ("fit_d16_single", 16, 4, 1, 2, [16 * 2000]),                     # per-node samples (c = 1)
    ("fit_d12", 12, 3, 3, 5, [12 * 900 + 4]),
]


@FIT_PATHS
@pytest.mark.parametrize("case", FIT_EDGE, ids=[c[0] for c in FIT_EDGE])
def test_fit_basis_edge_cases(gvq, oracle, case, fit_path):
    name, d, k, N, L, lens = case
    w = W.custom(name, 500 + d, d=d, k=k, N=N, L=L, layer_len=lens, layer_off=_gapped_offsets(lens))
    c = 1 if "single" in name else N
    hist = W.stored_gradients(w)
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda")
    mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    ctx.fit_basis(hist.cuda(), N, c, Ut, mu, ev)
    _check_fit(w, oracle, hist.numpy(), Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), N, c,
               tail_tol=FIT_TAIL_TOL[fit_path])


@FIT_PATHS
@pytest.mark.parametrize("d,k", [(128, 16), (32, 4)], ids=["tensor_core", "fp32_pipe"])
def test_fit_basis_with_a_mean_far_above_the_spread(gvq, oracle, d, k, fit_path):
    """Gradients whose mean is 50 standard deviations from zero, and different in the two halves of a layer:
    the covariance must not lose digits to the mean (the tensor-core path centres by a sampled point and corrects)."""
    lens = [d * 700, d * 150 + 4]
    w = W.custom("fit_big_mean", 77, d=d, k=k, N=4, L=5, layer_len=lens, layer_off=_gapped_offsets(lens))
    hist = W.stored_gradients(w)
    spread = float(hist[:, : lens[0]].std())
    hist[:, : lens[0] // 2] += 50.0 * spread
    hist[:, lens[0] // 2: lens[0]] -= 20.0 * spread
    hist[:, w.layer_off[1]: w.layer_off[1] + lens[1]] += 50.0 * spread
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda")
    mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    ctx.fit_basis(hist.cuda(), w.N, w.N, Ut, mu, ev)
    _check_fit(w, oracle, hist.numpy(), Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), w.N, w.N,
               tail_tol=FIT_TAIL_TOL[fit_path])


@pytest.mark.parametrize("fit_path", [0, 1], ids=["automatic", "rotations_kept"])
def test_fit_basis_resnet50_sampled_layers(gvq, oracle, fit_path):
    """Full-size refresh (L = 32, drifting factor); three layers re-fitted by the oracle.  (54 layers do not fit the
    GPU at once with the rotations kept, so the automatic choice is the values-and-subspace path.)"""
    w = W.resnet50()
    hist = W.stored_gradients(w, device="cuda")
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda")
    mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    sweeps = ctx.fit_basis(hist, w.N, w.N, Ut, mu, ev)
    assert all(0 < s < 30 for s in sweeps)
    G = Ut.cpu().numpy().astype(np.float64)
    assert np.abs(np.einsum("lkd,ljd->lkj", G, G) - np.eye(w.k)).max() <= 1e-5
    for l in (0, 1, 43):  # 7x7 stem (36 slices + tail), a 1x1 (16 slices), a 1x1 512->2048 layer
        m = w.layer_len[l]
        sub = W.custom("sub", 1, d=w.d, k=w.k, N=w.N, L=w.L, layer_len=[m])
        h = hist[:, w.layer_off[l]: w.layer_off[l] + m].contiguous().cpu().numpy()
        _check_fit(sub, oracle, h, Ut[l:l + 1].cpu().numpy(), mu[l:l + 1].cpu().numpy(), ev[l:l + 1].cpu().numpy(),
                   w.N, w.N, tail_tol=FIT_TAIL_TOL[fit_path])


@FIT_PATHS
@pytest.mark.parametrize("seed", range(8))
def test_fit_basis_random_layouts(gvq, oracle, seed, fit_path):
    """Seeded random layouts (ragged layers, empty ones, layers with fewer samples than d: rank-deficient covariances)
    through gvq_fit_basis on both eigen paths, every layer against the oracle."""
    rng = np.random.default_rng(2000 + seed)
    d, k = [(16, 4), (64, 8), (128, 16), (256, 32), (64, 16), (32, 4), (12, 3), (192, 32)][seed]
    N, L = int(rng.integers(1, 6)), int(rng.integers(1, 5))
    lens = []
    for _ in range(int(rng.integers(2, 6))):
        S = int(rng.choice([0, 1, 3, d // 2, d, 2 * d + 1, 700]))
        lens.append(S * d + (int(rng.integers(0, d)) if rng.integers(0, 2) else 0))
    lens.append(d * 400)
    w = W.custom(f"randfit{seed}", 950 + seed, d=d, k=k, N=N, L=L, layer_len=lens, layer_off=_gapped_offsets(lens))
    hist = W.stored_gradients(w)
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut = torch.full((w.n_layers, k, d), float("nan"), device="cuda")
    mu = torch.full((w.n_layers, d), float("nan"), device="cuda")
    ev = torch.full((w.n_layers, d), float("nan"), device="cuda")
    ctx.fit_basis(hist.cuda(), N, N, Ut, mu, ev)
    assert torch.isfinite(Ut).all() and torch.isfinite(mu).all() and torch.isfinite(ev).all()
    _check_fit(w, oracle, hist.numpy(), Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), N, N)


def _fit_layers_against_oracle(gvq, oracle, w, layers, fit_path, tail_tol):
    """Full-size fit of workload w on device-generated stored gradients; the given layers re-fitted by the oracle."""
    hist = W.stored_gradients(w, device="cuda")
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda")
    mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    sweeps = ctx.fit_basis(hist, w.N, w.N, Ut, mu, ev)
    assert all(0 < s < 30 for s in sweeps)
    G = Ut.cpu().numpy().astype(np.float64)
    assert np.abs(np.einsum("lkd,ljd->lkj", G, G) - np.eye(w.k)).max() <= 1e-5
    sub, flat, _ = _whole_layers(w, layers)
    h = hist[:, flat.cuda()].cpu().numpy()
    idx = list(layers)
    return _check_fit(sub, oracle, h, Ut.cpu().numpy()[idx], mu.cpu().numpy()[idx], ev.cpu().numpy()[idx], w.N, w.N,
                      tail_tol=tail_tol)


def test_fit_basis_vgg16_every_layer(gvq, oracle):
    """The VGG-16-shaped configuration's refresh at full size (L = 8), all 13 layers against the oracle."""
    w = W.vgg16()
    _fit_layers_against_oracle(gvq, oracle, w, range(w.n_layers), 0, FIT_TAIL_TOL[2])


def test_fit_basis_large_whole_layers(gvq, oracle):
    """The 100 M-entry configuration's refresh at full size (L = 8), five layers against the oracle."""
    free, _ = torch.cuda.mem_get_info()
    w = W.large()
    if free < (w.L + 1) * w.M * 4 + (4 << 30):
        pytest.skip("not enough free device memory for the stored gradients of the 100M-entry workload")
    _fit_layers_against_oracle(gvq, oracle, w, LARGE_WHOLE_LAYERS, 0, FIT_TAIL_TOL[2])


# stem, first bottleneck (1x1, 3x3, 1x1, projection), one 3x3 and one 1x1 of every later stage, the last block's
# 3x3 and 1x1, the FC layer
RESNET50_FIT_LAYERS = (0, 1, 2, 3, 4, 12, 13, 25, 27, 44, 46, 51, 52, 53)


def test_fit_basis_resnet50_many_layers(gvq, oracle):
    """The ResNet-50-shaped refresh (L = 32, drifting factor) on the default path, 14 of the 54 layers -- the stem,
    every stage, the FC layer -- against the oracle."""
    _fit_layers_against_oracle(gvq, oracle, W.resnet50(), RESNET50_FIT_LAYERS, 0, FIT_TAIL_TOL[2])


SHARD = [
    ("shard_d256", 256, 32, 4, 6, [256 * 300 + 8, 256 * 700, 100]),        # tensor-core covariance, a layer without a slice
    ("shard_d128", 128, 16, 3, 5, [128 * 900 + 17, 128 * 40]),
    ("shard_d16", 16, 4, 4, 8, [16 * 1024]),                                # FP32-pipe covariance
    ("shard_d12", 12, 3, 2, 4, [12 * 900 + 4, 12 * 33]),
]


@FIT_PATHS
@pytest.mark.parametrize("case", SHARD, ids=[c[0] for c in SHARD])
def test_fit_from_the_moments_of_two_participants(gvq, oracle, case, fit_path):
    """The stored gradients split between two participants (here: two calls on one GPU): a common centre from the
    first one's samples, each one's moments about it, their sum, the fit from the sum -- against the oracle's fit of
    all samples at once (same bars as gvq_fit_basis) and against the oracle's own moments."""
    name, d, k, N, L, lens = case
    w = W.custom(name, 600 + d, d=d, k=k, N=N, L=L, layer_len=lens, layer_off=_gapped_offsets(lens))
    hist = W.stored_gradients(w)
    hist += 5.0 * float(hist.std())                       # a mean well away from zero
    hist_dev = hist.cuda()
    halves = [hist_dev[: L // 2].contiguous(), hist_dev[L // 2:].contiguous()]
    ctx = gvq.Context(w)
    ctx.set_fit_path(fit_path)
    centre = torch.full((w.n_layers, d), float("nan"), device="cuda")
    ctx.fit_centre(halves[0], centre)
    parts = []
    for h in halves:
        m = torch.full((ctx.layout.fit_moments_count(),), float("nan"), dtype=torch.float64, device="cuda")
        ctx.fit_moments(h, centre, m)
        parts.append(m)
    ctx.device_status()
    c_np = centre.cpu().numpy()
    for h, m in zip(halves, parts):                       # one participant's moments against their definition
        want = oracle.fit_moments(w, h.cpu().numpy(), c_np)
        got = m.cpu().numpy().reshape(w.n_layers, -1)
        assert np.array_equal(got[:, 0], want[:, 0])
        for l in range(w.n_layers):
            scale = np.abs(want[l, 1 + d:]).max() + 1e-30
            # fp32 partial sums (the tensor-core accumulator rounds toward zero: ~2e-6 of the largest entry)
            assert np.abs(got[l, 1 + d:] - want[l, 1 + d:]).max() <= 1e-5 * scale, f"second moments layer {l}"
            assert np.abs(got[l, 1:1 + d] - want[l, 1:1 + d]).max() <= 1e-5 * (np.abs(want[l, 1:1 + d]).max() + np.sqrt(scale)), l
    Ut = torch.full((w.n_layers, k, d), float("nan"), device="cuda")
    mu = torch.full((w.n_layers, d), float("nan"), device="cuda")
    ev = torch.full((w.n_layers, d), float("nan"), device="cuda")
    sweeps = ctx.fit_from_moments(parts[0] + parts[1], centre, N, N, Ut, mu, ev)
    assert all(0 < s < 30 for s in sweeps)
    _check_fit(w, oracle, hist.numpy(), Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), N, N)
    # and the one-GPU call on all samples gives the same fit
    Ut1 = torch.empty_like(Ut); mu1 = torch.empty_like(mu); ev1 = torch.empty_like(ev)
    ctx.fit_basis(hist_dev, N, N, Ut1, mu1, ev1)
    for l in range(w.n_layers):
        assert np.abs((ev1[l] - ev[l]).cpu().numpy()).max() <= 1e-5 * max(float(ev1[l, 0]), 1e-30)
        if w.layer_len[l] >= d:
            assert subspace_angle(Ut[l].cpu().numpy(), Ut1[l].cpu().numpy()) <= 1e-4


def test_select_k_agrees_between_the_fit_paths_and_with_the_oracle(gvq, oracle):
    """Eq. 6 on the eigenvalues of both fit paths, on spectra whose mass ratio sits near the threshold: the k chosen
    from the library's eigenvalues is the oracle's, whichever path produced them."""
    d, k, N, L = 64, 8, 3, 6
    w = W.custom("selk", 71, d=d, k=k, N=N, L=L, layer_len=[d * 400, d * 150 + 8, d * 20])
    hist = W.stored_gradients(w)
    # a slowly decaying extra component in layer 1, so that the ratio crosses 1 - lambda inside the tail
    g = torch.Generator().manual_seed(9)
    a, m = w.layer_off[1], (w.layer_len[1] // d) * d
    scale = torch.logspace(0.5, -2.0, d)
    hist[:, a:a + m] += (torch.randn((L, m // d, d), generator=g) * scale).reshape(L, m)
    o_Ut, o_mu, o_ev, _ = oracle.fit_basis(w, hist.numpy(), N=N, samples_are_sums_of=N)
    picks = {}
    for fit_path in (1, 2):
        ctx = gvq.Context(w)
        ctx.set_fit_path(fit_path)
        Ut = torch.empty((w.n_layers, k, d), device="cuda"); mu = torch.empty((w.n_layers, d), device="cuda")
        ev = torch.empty((w.n_layers, d), device="cuda")
        ctx.fit_basis(hist.cuda(), N, N, Ut, mu, ev)
        picks[fit_path] = ev.cpu()
    checked = 0
    for l in range(w.n_layers):
        total = o_ev[l].sum()
        # thresholds that put the cut inside the spectrum, each with a clear margin to the next eigenvalue
        for kk in (2, k - 1, k, k + 3, d // 2, d - 5):
            head, nxt = o_ev[l][:kk].sum() / total, o_ev[l][: kk + 1].sum() / total
            if nxt - head < 1e-4:
                continue           # the ratio moves by less than the bar on the eigenvalues: any of the two is right
            lam = 1.0 - 0.5 * (head + nxt)
            want = oracle.select_k(o_ev[l], lam)
            assert want == kk + 1
            for fit_path in (1, 2):
                assert gvq.select_k(picks[fit_path][l], lam) == want, (l, kk, fit_path)
            checked += 1
    assert checked >= 8


# ------------------------------------------------------------------------------ error paths (host side only)
@pytest.mark.parametrize("name,warm", [("resnet32", False), ("resnet32", True), ("sub_d128k16", False), ("sub_d256k32", True),
                                       ("sub_rank_deficient", False), ("sub_odd_k", False)])
def test_refresh_basis_by_subspace_iteration(gvq, oracle, name, warm):
    """The cheap refresh against the definition it approximates: the k leading eigenpairs of the covariance (the
    oracle's full fit).  The synthetic spectra have a gap of ~1e2 after k, so 8 rounds from a random start (3 from the
    previous basis) are far below the bar: subspace angle 1e-4, eigenvalues 1e-5 of the largest, trace 1e-5."""
    if name == "resnet32":
        w = W.resnet32()
    elif name == "sub_d128k16":
        w = W.custom(name, 61, d=128, k=16, N=4, L=6, layer_len=[128 * 300, 128 * 90 + 40, 128 * 700])
    elif name == "sub_d256k32":
        w = W.custom(name, 62, d=256, k=32, N=4, L=6, layer_len=[256 * 200, 256 * 330 + 8])
    elif name == "sub_odd_k":
        w = W.custom(name, 64, d=64, k=5, N=3, L=8, layer_len=[64 * 150, 64 * 40])
    else:
        w = W.custom(name, 63, d=64, k=8, N=3, L=4, layer_len=[64 * 100, 64 * 30])
    hist = W.stored_gradients(w)
    if name == "sub_rank_deficient":      # layer 1: every sample a multiple of one vector plus a constant: rank 1 < k
        a, m = w.layer_off[1], w.layer_len[1]
        v = torch.linspace(-1, 1, w.d)
        coef = torch.arange(hist.shape[0] * (m // w.d), dtype=torch.float32).reshape(hist.shape[0], m // w.d, 1)
        hist[:, a:a + m] = (coef * v + 0.5).reshape(hist.shape[0], m)
    ctx = gvq.Context(w)
    Ut = torch.full((w.n_layers, w.k, w.d), float("nan"), device="cuda")
    mu = torch.full((w.n_layers, w.d), float("nan"), device="cuda")
    ev = torch.full((w.n_layers, w.k), float("nan"), device="cuda")
    tr = torch.full((w.n_layers,), float("nan"), device="cuda")
    if warm:    # the previous basis: the exact one, rotated a little towards a random one
        o_prev, _, _, _ = oracle.fit_basis(w, hist.numpy(), N=w.N, samples_are_sums_of=w.N)
        g = torch.Generator().manual_seed(5)
        Ut.copy_(torch.as_tensor(o_prev, dtype=torch.float32) + 0.05 * torch.randn(o_prev.shape, generator=g))
    ctx.refresh_basis(hist.cuda(), w.N, w.N, Ut, mu, ev, tr, iters=3 if warm else 8, warm_start=warm)
    o_Ut, o_mu, o_ev, _ = oracle.fit_basis(w, hist.numpy(), N=w.N, samples_are_sums_of=w.N)
    Ut_g, mu_g, ev_g, tr_g = Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), tr.cpu().numpy()
    for l in range(w.n_layers):
        G = Ut_g[l].astype(np.float64)
        assert np.abs(G @ G.T - np.eye(w.k)).max() <= 1e-5, f"orthonormality layer {l}"
        lam_max = max(o_ev[l, 0], 1e-30)
        assert np.abs(ev_g[l] - o_ev[l, : w.k]).max() <= 1e-5 * lam_max, f"eigenvalues layer {l}"
        assert abs(tr_g[l] - o_ev[l].sum()) <= 1e-5 * max(o_ev[l].sum(), 1e-30), f"trace layer {l}"
        assert np.all(np.diff(ev_g[l]) <= 0)
        assert np.allclose(mu_g[l], o_mu[l], rtol=1e-5, atol=1e-6 * (np.abs(o_mu[l]).max() + 1e-30))
        if o_ev[l, w.k - 1] > 10 * o_ev[l, w.k]:
            assert subspace_angle(G, o_Ut[l]) <= 1e-4, f"subspace layer {l}"
            big = np.abs(G).argmax(axis=1)
            assert np.all(G[np.arange(w.k), big] > 0)
        elif name == "sub_rank_deficient" and l == 1:
            # rank 1: the leading vector is the direction, the others any orthonormal completion
            assert subspace_angle(G[:1], o_Ut[l][:1]) <= 1e-4 and np.all(ev_g[l, 1:] <= 1e-5 * lam_max)


def test_reuse_factor_first_slice_sampling(gvq, oracle):
    """Section 3's compressor reuse factor s: one compressor per s consecutive slices, fitted from the FIRST slice
    of the group only.  Both are layouts of this library: a group is a "layer" of s slices for the streaming
    calls, and its first slice is a "layer" of one slice for the fit; the (Ut, mu) arrays are the same."""
    d, k, N, L, s_reuse, S = 16, 4, 3, 40, 64, 230
    wb = W.custom("reuse_base", 55, d=d, k=k, N=N, L=L, layer_len=[d * S])
    starts = list(range(0, S, s_reuse))
    g_len = [min(s_reuse, S - a) * d for a in starts]
    wg = W.custom("reuse_groups", 56, d=d, k=k, N=N, L=L, layer_len=g_len, layer_off=[a * d for a in starts])
    wf = W.custom("reuse_first", 57, d=d, k=k, N=N, L=L, layer_len=[d] * len(starts), layer_off=[a * d for a in starts])
    hist = W.stored_gradients(wb)
    ctx_f = gvq.Context(wf)
    Ut = torch.full((len(starts), k, d), float("nan"), device="cuda")
    mu = torch.full((len(starts), d), float("nan"), device="cuda")
    ev = torch.full((len(starts), d), float("nan"), device="cuda")
    ctx_f.fit_basis(hist.cuda(), N, N, Ut, mu, ev)
    _check_fit(wf, oracle, hist.numpy(), Ut.cpu().numpy(), mu.cpu().numpy(), ev.cpu().numpy(), N, N, tail_tol=FIT_TAIL_TOL[0])
    # the same arrays drive the streaming path over the groups
    g = [t.numpy() for t in W.node_gradients(wb, iteration=L)]
    ctx, s_sum, g_hat, _ = _run_stream(gvq, wg, [_dev(x) for x in g], Ut, mu)
    _check_stream(wg, oracle, g, Ut.cpu().numpy(), mu.cpu().numpy(), s_sum, g_hat)
    # and the compressor of a group's first slice serves the rest of the group (spatial consistency): small loss
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    assert rel_l2(g_hat.cpu().numpy(), gsum) < 0.1


RAW4 = [
    ("raw4_d256", 256, 32, 4, [256 * 300 + 100, 256 * 5, 30]),
    ("raw4_d64", 64, 8, 3, [64 * 700 + 20]),
    ("raw4_d16", 16, 4, 5, [16 * 257 + 5, 7, 16 * 33]),
    ("raw4_d12", 12, 3, 2, [12 * 77 + 8]),
    ("raw4_d192", 192, 32, 2, [192 * 140]),
    ("raw4_d512", 512, 24, 2, [512 * 65 + 4]),
]


@pytest.mark.parametrize("case", RAW4, ids=[c[0] for c in RAW4])
def test_quantize_raw4_bit_exact(gvq, oracle, case):
    """The 4-bit quantizer on raw slices: packed levels and norms bit for bit, the aggregate of the dequantised
    gradients to fp32 rounding, tails as the plain fp32 sum in node order."""
    name, d, k, N, lens = case
    w = W.custom(name, 700 + d, d=d, k=k, N=N, L=1, layer_len=lens, layer_off=_gapped_offsets(lens))
    g = [t.numpy() for t in W.node_gradients(w)]
    g[0][w.layer_off[0]:w.layer_off[0] + d] = 0.0          # a zero slice: norm 0, all levels 0
    g_dev = [_dev(x) for x in g]
    ctx = gvq.Context(w)
    levels, seed = 7, 20181103
    q4s, nss, o_q4, o_ns = [], [], [], []
    for n in range(N):
        q4 = torch.full((ctx.S, d // 2), 0xEE, dtype=torch.uint8, device="cuda")
        ns = torch.full((ctx.S,), float("nan"), device="cuda")
        ctx.quantize_raw4(g_dev[n], levels, seed, n, q4, ns)
        a, b = oracle.quantize_raw4(w, g[n], levels, seed, n)
        assert np.array_equal(q4.cpu().numpy(), a), f"levels node {n}"
        assert np.array_equal(ns.cpu().numpy(), b), f"norms node {n}"
        q4s.append(q4); nss.append(ns); o_q4.append(a); o_ns.append(b)
    assert np.all(o_q4[0][0] == 0) and o_ns[0][0] == 0.0
    out = torch.full((w.M,), float("nan"), device="cuda")
    ctx.dequantize_raw4_aggregate(q4s, nss, g_dev, levels, out)
    want = oracle.dequantize_raw4_aggregate(w, o_q4, o_ns, g, levels, w.M)
    got = out.cpu().numpy()
    assert np.array_equal(np.isnan(got), np.isnan(want))
    cov = ~np.isnan(want)
    assert rel_l2(got[cov], want[cov]) <= 1e-6
    for l in range(w.n_layers):
        _, _, (ta, tb) = layer_slices(w, l)
        if tb > ta:
            seq = g[0][ta:tb].copy()
            for n in range(1, N):
                seq = seq + g[n][ta:tb]
            assert np.array_equal(got[ta:tb], seq)
    # the single-launch form is bit-identical, with and without the per-node outputs
    out2 = torch.full((w.M,), float("nan"), device="cuda")
    q2 = [torch.full((ctx.S, d // 2), 0xEE, dtype=torch.uint8, device="cuda") for _ in range(N)]
    n2 = [torch.full((ctx.S,), float("nan"), device="cuda") for _ in range(N)]
    ctx.quantize_raw4_aggregate(g_dev, levels, seed, out2, q2, n2)
    assert torch.equal(torch.nan_to_num(out2, nan=-7.0), torch.nan_to_num(out, nan=-7.0))
    assert all(torch.equal(a, b) for a, b in zip(q2, q4s)) and all(torch.equal(a, b) for a, b in zip(n2, nss))
    out3 = torch.full((w.M,), float("nan"), device="cuda")
    ctx.quantize_raw4_aggregate(g_dev, levels, seed, out3)
    assert torch.equal(torch.nan_to_num(out3, nan=-7.0), torch.nan_to_num(out, nan=-7.0))


@pytest.mark.parametrize("F,D,H,Wd", [(64, 3, 7, 7), (16, 16, 3, 3), (256, 64, 1, 1), (5, 3, 2, 7), (1, 1, 1, 1),
                                       (33, 65, 3, 3), (512, 512, 3, 3)])
def test_flatten_order_bit_exact(gvq, oracle, F, D, H, Wd):
    """The layer permutation of Section 2 and its inverse, bit for bit against the oracle (sampled for the
    largest layer, where the oracle's triple loop is slow)."""
    X = H * Wd
    ctx = gvq.Context(W.tiny())
    g = torch.Generator().manual_seed(F * 1000 + D)
    fw = torch.randn((F, D, X), generator=g)
    flat = torch.full((X, D, F), float("nan"), device="cuda")
    back = torch.full((F, D, X), float("nan"), device="cuda")
    ctx.flatten_layer(fw.cuda(), flat, F, D, X)
    ctx.unflatten_layer(flat, back, F, D, X)
    torch.cuda.synchronize()
    assert torch.equal(back.cpu(), fw)
    if F * D * X <= 1 << 20:
        assert np.array_equal(flat.cpu().numpy(), oracle.flatten(fw.numpy()))
    else:   # every entry against the index formula of the definition (vectorised), plus an oracle block
        want = fw.permute(2, 1, 0).contiguous()
        assert torch.equal(flat.cpu(), want)
        sub = fw[:40, :24].contiguous()
        assert np.array_equal(oracle.flatten(sub.numpy()), flat.cpu().numpy()[:, :24, :40])


def test_the_papers_iteration_plan_end_to_end(gvq):
    """Section 3's plan on synthetic gradients, driven by the library alone: L_t iterations aggregate 4-bit quantized
    gradients and store the aggregates as PCA samples; a fit; compressed iterations watched by the Eq. 7 monitor;
    when the gradients' subspace changes the majority rule ends the compressed phase."""
    w = W.custom("plan", 88, d=128, k=16, N=4, L=1, layer_len=[128 * 500, 128 * 260 + 40])
    w2 = W.custom("plan_moved", 89, d=128, k=16, N=4, L=1, layer_len=w.layer_len)   # another factor: a moved subspace
    ctx = gvq.Context(w)
    L_t, L_c = 6, 8
    sch = gvq.Schedule(L_t, L_c, w.N, 0.05)
    hist = torch.zeros((L_t, w.M), device="cuda")
    Ut = torch.empty((w.n_layers, w.k, w.d), device="cuda"); mu = torch.empty((w.n_layers, w.d), device="cuda")
    ev = torch.empty((w.n_layers, w.d), device="cuda")
    s_sum = torch.empty((ctx.S, w.k), device="cuda"); g_hat = torch.zeros(w.M, device="cuda")
    mon = torch.empty((w.n_layers, 2, w.N), dtype=torch.float64, device="cuda")
    q4 = [torch.empty((ctx.S, w.d // 2), dtype=torch.uint8, device="cuda") for _ in range(w.N)]
    ns = [torch.empty((ctx.S,), device="cuda") for _ in range(w.N)]
    log, stored, rel_err = [], 0, []
    for it in range(L_t + L_c + 2):
        moved = it >= L_t + 4
        g = [W.node_gradient(w2 if moved else w, n, iteration=it, device="cuda") for n in range(w.N)]
        exact = torch.stack(g).double().sum(0)
        if sch.phase == gvq.PHASE_COLLECT:
            for n in range(w.N):
                ctx.quantize_raw4(g[n], 7, 1234 + it, n, q4[n], ns[n])
            ctx.dequantize_raw4_aggregate(q4, ns, g, 7, hist[stored])
            stored += 1
            action = sch.step()
        else:
            ctx.compress_aggregate_monitored(g, Ut, mu, s_sum, mon)
            ctx.decompress(s_sum, Ut, mu, g, w.N, g_hat)
            rel_err.append(float((g_hat.double() - exact).norm() / exact.norm()))
            action = sch.step(mon.cpu())
        log.append(action)
        if action == gvq.ACT_FIT:
            ctx.fit_basis(hist, w.N, w.N, Ut, mu, ev)
        if action == gvq.ACT_RESTART:
            break
    assert log[:L_t] == [gvq.ACT_NONE] * (L_t - 1) + [gvq.ACT_FIT]
    # compressed iterations on the fitted subspace lose little (4-bit samples cost some accuracy of the basis) ...
    assert all(e < 0.12 for e in rel_err[:4]), rel_err
    # ... and the first iteration on the moved subspace puts every node over the threshold
    assert log[-1] == gvq.ACT_RESTART and len(log) == L_t + 5 and sch.nodes_over == w.N
    assert rel_err[-1] > 0.5


def test_error_codes(gvq):
    w = W.tiny()
    ctx = gvq.Context(w)
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g = [torch.zeros(w.M + 4, device="cuda") for _ in range(w.N)]
    s = torch.empty((ctx.S, w.k), device="cuda")
    with pytest.raises(gvq.GvqError) as e:  # misaligned input
        ctx.compress_aggregate([x[1:] for x in g], Ut, mu, s)
    assert e.value.status == 3
    with pytest.raises(gvq.GvqError) as e:  # output aliases a per-node output
        ctx.compress_aggregate(g, Ut, mu, s, [s] * w.N)
    assert e.value.status == 2
    ctx.set_workspace(None)
    with pytest.raises(gvq.GvqError) as e:  # fit without a workspace
        gvq._check(gvq.lib().gvq_fit_basis(ctx._h, g[0].data_ptr(), w.M, 1, w.N, w.N, Ut.data_ptr(), mu.data_ptr(),
                                           mu.data_ptr(), None), "gvq_fit_basis")
    assert e.value.status == 5
    with pytest.raises(gvq.GvqError) as e:
        ctx.quantize(s, 128, 1, 0, torch.empty((ctx.S, w.k), dtype=torch.int8, device="cuda"),
                     torch.empty(ctx.S, device="cuda"))
    assert e.value.status == 2
    # the context is still usable after the refusals
    ctx.compress_aggregate([x[: w.M] for x in g], Ut, mu, s)
    torch.cuda.synchronize()
