"""Algorithm 1 on one GPU: the exchange-buffer entry points of the C ABI, and the ring's participants stepped in
lock-step in one process (same kernels and schedule as the multi-process ring, copies in place of the links),
against the oracle's direct evaluation of Eq. 3-5 and its node-by-node simulation of the algorithm."""
import ctypes

import numpy as np
import pytest
import torch

from paper_1811_03617_b200 import workloads as W
from util import layer_slices, rel_l2

pytestmark = pytest.mark.gpu

TOL = 1e-5


@pytest.fixture(scope="module")
def gvq():
    from paper_1811_03617_b200 import gvq as _gvq
    _gvq.lib()
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    return _gvq


def _ragged(d, k, N, ident):
    return W.custom(f"ring_d{d}k{k}", ident, d=d, k=k, N=N, L=1,
                    layer_len=[d * 7 + 4, 8, d * 300, d * 3 + 4, 0, d * 131, 12, d * 129 + d // 2])


CASES = [("tiny", lambda: W.tiny(), 4), ("resnet32", lambda: W.resnet32(), 4),
         ("ragged_fp32_pipe", lambda: _ragged(16, 4, 6, 171), 3), ("ragged_tensor_core", lambda: _ragged(128, 16, 8, 172), 4)]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_partial_accumulate_exchanged_equals_the_one_gpu_path(gvq, oracle, case):
    """N nodes in `groups` groups: each group's partial buffer (mean scaled by 1 / N), added up, decompressed."""
    _, make, groups = case
    w = make()
    g = W.node_gradients(w)
    Ut, mu = W.random_basis(w)
    g_dev, Ut_d, mu_d = [x.cuda() for x in g], Ut.cuda(), mu.cuda()
    ctx = gvq.Context(w)
    nx = ctx.layout.exchange_floats()
    assert nx == w.S * w.k + w.tail_entries
    per = -(-w.N // groups)
    x_acc = None
    for a in range(0, w.N, per):
        x = torch.full((max(nx, 4),), float("nan"), device="cuda")
        ctx.compress_aggregate_partial(g_dev[a:a + per], w.N, Ut_d, mu_d, x)
        if x_acc is None:
            x_acc = x
        else:
            ctx.exchange_accumulate(x_acc, x)
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    ctx.decompress_exchanged(x_acc, Ut_d, mu_d, g_hat)
    ctx.device_status()
    g_np = [x.numpy() for x in g]
    o_s, o_g = oracle.pipeline(w, g_np, Ut.numpy(), mu.numpy())
    xs = x_acc.cpu().numpy()
    assert rel_l2(xs[: w.S * w.k], o_s) <= TOL
    got = g_hat.cpu().numpy()
    covered = np.zeros(w.M, dtype=bool)
    p = w.S * w.k
    for l in range(w.n_layers):
        (a, b), (sa, sb), (ta, tb) = layer_slices(w, l)
        covered[a:tb] = True
        if sb > sa:
            assert rel_l2(got[a:b], o_g[a:b]) <= TOL, f"g_hat layer {l}"
        if tb > ta:
            assert np.allclose(got[ta:tb], o_g[ta:tb], rtol=1e-5, atol=1e-5), f"tail layer {l}"
            assert np.array_equal(got[ta:tb], xs[p:p + tb - ta])       # tails sit in layer order behind the slices
            p += tb - ta
    assert p == nx
    assert np.all(np.isnan(got[~covered]))


RING = [("tiny_w4", lambda: W.tiny(), 4, 1), ("resnet32_w8", lambda: W.resnet32(), 8, 1),
        ("resnet32_w3_two_nodes_each", lambda: W.custom("r32x6", 173, d=64, k=8, N=6, L=1, layer_len=W.resnet32().layer_len), 3, 2),
        ("ragged_fp32_pipe_w5", lambda: _ragged(16, 4, 5, 174), 5, 1),
        ("ragged_tensor_core_w4", lambda: _ragged(128, 16, 8, 175), 4, 2),
        ("resnet50_full_size_w4", lambda: W.custom("r50x4", 178, d=256, k=32, N=4, L=1, layer_len=W.resnet50().layer_len), 4, 1),
        ("more_participants_than_slices", lambda: W.custom("few", 176, d=16, k=4, N=6, L=1, layer_len=[16 * 2 + 4, 16, 8]), 6, 1)]


@pytest.mark.parametrize("case", RING, ids=[c[0] for c in RING])
def test_ring_participants_in_lock_step(gvq, oracle, case):
    from paper_1811_03617_b200 import ring
    _, make, world, n_local = case
    w = make()
    assert w.N == world * n_local
    g = W.node_gradients(w)
    Ut, mu = W.random_basis(w)
    g_dev, Ut_d, mu_d = [x.cuda() for x in g], Ut.cuda(), mu.cuda()
    engine = ring.CudaSegmentEngine(w, world)
    lr = ring.LocalRing(lambda: engine, world)
    g_hat = [torch.full((w.M,), float("nan"), device="cuda") for _ in range(world)]
    lr.run([g_dev[n * n_local:(n + 1) * n_local] for n in range(world)], w.N, Ut_d, mu_d, g_hat)
    for c in engine.ctx:
        if c is not None:
            c.device_status()
    g_np = [x.numpy() for x in g]
    _, o_g = oracle.pipeline(w, g_np, Ut.numpy(), mu.numpy())
    covered = np.zeros(w.M, dtype=bool)
    for l in range(w.n_layers):
        covered[w.layer_off[l]:w.layer_off[l] + w.layer_len[l]] = True
    got0 = g_hat[0].cpu().numpy()
    for l in range(w.n_layers):
        (a, b), _, (ta, tb) = layer_slices(w, l)
        if b > a:
            assert rel_l2(got0[a:b], o_g[a:b]) <= TOL, f"layer {l}"
        if tb > ta:
            assert np.allclose(got0[ta:tb], o_g[ta:tb], rtol=1e-5, atol=1e-5)
    assert rel_l2(got0[covered], o_g[covered]) <= TOL
    assert np.all(np.isnan(got0[~covered]))
    # every participant decompresses the same aggregated segments: identical bits on all of them
    for n in range(1, world):
        assert torch.equal(g_hat[n][torch.from_numpy(covered).cuda()], g_hat[0][torch.from_numpy(covered).cuda()])
    # the messages are Algorithm 1's: sizes per node as in the oracle's simulation, d / k below a raw ring
    assert sum(p.floats_sent for p in lr.nodes) == 2 * (world - 1) * (w.S * w.k + w.tail_entries)
    if n_local == 1:
        _, sent = oracle.ring_allreduce(w, g_np, Ut.numpy(), mu.numpy())
        assert [p.floats_sent for p in lr.nodes] == sent
    engine.close()


def test_single_process_collective_variant(gvq, oracle):
    """allreduce_compressed without a process group: partial buffer -> (no exchange) -> decompression."""
    from paper_1811_03617_b200 import ring
    w = W.resnet32()
    g = W.node_gradients(w)
    Ut, mu = W.random_basis(w)
    ctx = gvq.Context(w)
    x = torch.empty(ctx.layout.exchange_floats(), device="cuda")
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    ring.allreduce_compressed(ctx, [t.cuda() for t in g], w.N, Ut.cuda(), mu.cuda(), x, g_hat)
    ctx.device_status()
    _, o_g = oracle.pipeline(w, [t.numpy() for t in g], Ut.numpy(), mu.numpy())
    assert rel_l2(g_hat.cpu().numpy(), o_g) <= TOL


def test_exchange_entry_points_at_full_size(gvq):
    """The ResNet-50-shaped layout at full size, four nodes in two groups: partial buffers added up and decompressed
    give what the one-GPU calls give on the same gradients (tensor-core kernels on both routes; the sum over nodes is
    taken in another order, hence 1e-6 and not equality)."""
    base = W.resnet50()
    w = W.custom("ring_full", 177, d=base.d, k=base.k, N=4, L=1, layer_len=base.layer_len)
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g = [W.node_gradient(w, n, device="cuda") for n in range(w.N)]
    ctx = gvq.Context(w)
    s_sum = torch.empty((ctx.S, w.k), device="cuda")
    want = torch.full((w.M,), float("nan"), device="cuda")
    ctx.compress_aggregate(g, Ut, mu, s_sum)
    ctx.decompress(s_sum, Ut, mu, g, w.N, want)
    nx = ctx.layout.exchange_floats()
    xa = torch.full((nx,), float("nan"), device="cuda")
    xb = torch.full((nx,), float("nan"), device="cuda")
    ctx.compress_aggregate_partial(g[:2], w.N, Ut, mu, xa)
    ctx.compress_aggregate_partial(g[2:], w.N, Ut, mu, xb)
    ctx.exchange_accumulate(xa, xb)
    got = torch.full((w.M,), float("nan"), device="cuda")
    ctx.decompress_exchanged(xa, Ut, mu, got)
    ctx.device_status()
    assert torch.isfinite(xa).all()
    assert rel_l2(xa[: ctx.S * w.k].cpu().numpy(), s_sum.flatten().cpu().numpy()) <= 1e-6
    covered = torch.zeros(w.M, dtype=torch.bool, device="cuda")
    for o, m in zip(w.layer_off, w.layer_len):
        covered[o:o + m] = True
    assert rel_l2(got[covered].cpu().numpy(), want[covered].cpu().numpy()) <= 1e-6
    for l in range(w.n_layers):
        _, _, (ta, tb) = layer_slices(w, l)
        if tb > ta:     # (g0 + g1) + (g2 + g3) against ((g0 + g1) + g2) + g3: the same to rounding, not bit for bit
            assert torch.allclose(got[ta:tb], want[ta:tb], rtol=1e-6, atol=1e-6)


def test_exchange_entry_points_refuse_bad_arguments(gvq):
    w = W.tiny()
    ctx = gvq.Context(w)
    Ut_t, mu_t = W.random_basis(w)
    Ut, mu = Ut_t.cuda(), mu_t.cuda()
    g = [torch.zeros(w.M + 4, device="cuda") for _ in range(2)]
    x = torch.zeros(ctx.layout.exchange_floats() + 4, device="cuda")
    with pytest.raises(gvq.GvqError) as e:      # more local gradients than the job has nodes
        ctx.compress_aggregate_partial([t[: w.M] for t in g], 1, Ut, mu, x)
    assert e.value.status == 2
    with pytest.raises(gvq.GvqError) as e:      # misaligned exchange buffer
        ctx.compress_aggregate_partial([t[: w.M] for t in g], 4, Ut, mu, x[1:])
    assert e.value.status == 3
    with pytest.raises(gvq.GvqError) as e:      # a buffer added to itself
        ctx.exchange_accumulate(x, x)
    assert e.value.status == 2
    with pytest.raises(gvq.GvqError) as e:
        gvq._check(gvq.lib().gvq_decompress_exchanged(ctx._h, None, Ut.data_ptr(), mu.data_ptr(), g[0].data_ptr()),
                   "gvq_decompress_exchanged")
    assert e.value.status == 1
    ctx.compress_aggregate_partial([t[: w.M] for t in g], 4, Ut, mu, x)     # still usable
    ctx.device_status()


def test_packed_exchange_with_per_layer_k(gvq, oracle):
    """Eq. 6 layer by layer: with the basis masked to k_l rows per layer, the exchange buffer is packed to
    sum_l S_l k_l + T floats, two participants' packed buffers are added (what a collective does), and the unpacked
    sum decompresses to what the oracle computes with k_l columns per layer."""
    from paper_1811_03617_b200 import ring
    lens = [128 * 259, 128 * 3 + 100, 128 * 140, 60, 128 * 64]
    w = W.custom("packed_k", 93, d=128, k=16, N=4, L=1, layer_len=lens)
    ks = [16, 5, 0, 7, 9]
    Ut_t, mu_t = W.random_basis(w)
    g = [t.numpy() for t in W.node_gradients(w)]
    g_dev = [torch.as_tensor(x).cuda() for x in g]
    ctx = gvq.Context(w)
    Ut_dev, mu_dev = Ut_t.cuda(), mu_t.cuda()
    ctx.mask_basis(Ut_dev, ks)
    ctx.set_layer_k(ks)
    n_full, n_packed = ctx.layout.exchange_floats(), ctx.layout.packed_floats(ks)
    S_l = [m // w.d for m in lens]
    assert n_packed == sum(a * b for a, b in zip(S_l, ks)) + w.tail_entries and n_packed < n_full
    halves = [g_dev[:2], g_dev[2:]]
    xs, ps = [], []
    for part in halves:
        x = torch.full((n_full,), float("nan"), device="cuda")
        xp = torch.full((n_packed,), float("nan"), device="cuda")
        ctx.compress_aggregate_partial(part, w.N, Ut_dev, mu_dev, x)
        ctx.exchange_pack(x, xp)
        xs.append(x); ps.append(xp)
    ctx.device_status()
    # the packed buffer is the kept coordinates, layer after layer, then the tails -- bit for bit
    x0 = xs[0].cpu().numpy()
    want, row = [], 0
    for S, kl in zip(S_l, ks):
        want.append(x0[row * w.k:(row + S) * w.k].reshape(S, w.k)[:, :kl].ravel())
        row += S
    want.append(x0[row * w.k:])
    assert np.array_equal(ps[0].cpu().numpy(), np.concatenate(want))
    # unpack restores the buffer (the dropped coordinates were exact zeros)
    back = torch.full((n_full,), float("nan"), device="cuda")
    ctx.exchange_unpack(ps[0], back)
    assert torch.equal(back, xs[0])
    # the collective's sum on packed buffers, then Eq. 5
    total = ps[0] + ps[1]
    x_sum = torch.full((n_full,), float("nan"), device="cuda")
    g_hat = torch.full((w.M,), float("nan"), device="cuda")
    ctx.exchange_unpack(total, x_sum)
    ctx.decompress_exchanged(x_sum, Ut_dev, mu_dev, g_hat)
    ctx.device_status()
    got = g_hat.cpu().numpy()
    Ut, mu = Ut_t.numpy(), mu_t.numpy()
    for l, kl in enumerate(ks):
        a, m = w.layer_off[l], lens[l]
        S = m // w.d
        seg = [x[a:a + m] for x in g]
        if S > 0 and kl > 0:
            wl = W.custom(f"packed_l{l}", 1, d=w.d, k=kl, N=w.N, L=1, layer_len=[m], layer_off=[0])
            Ul, ml = np.ascontiguousarray(Ut[l:l + 1, :kl]), mu[l:l + 1]
            o_s = oracle.aggregate([oracle.compress(wl, x, Ul, ml, w.N) for x in seg])
            o_g = oracle.decompress(wl, o_s, Ul, ml, seg, w.N, m)
            assert rel_l2(got[a:a + m], o_g) <= 1e-5, l
        elif S > 0:
            assert np.allclose(got[a:a + S * w.d].reshape(S, w.d), mu[l][None, :], rtol=0, atol=1e-6)
        tail = sum(x[S * w.d:].astype(np.float64) for x in seg)
        assert np.allclose(got[a + S * w.d:a + m], tail, rtol=1e-6, atol=1e-6)
    # the same through the one-collective helper (world 1: no collective), and back to all k
    g_hat2 = torch.full((w.M,), float("nan"), device="cuda")
    ring.allreduce_compressed(ctx, g_dev, w.N, Ut_dev, mu_dev, x_sum, g_hat2, x_packed=total)
    ctx.device_status()
    assert rel_l2(g_hat2.cpu().numpy()[: w.M], got) <= 1e-6
    ctx.set_layer_k(None)
    assert gvq.lib().gvq_set_layer_k(ctx._h, (ctypes.c_int32 * w.n_layers)(17, 0, 0, 0, 0)) == 2
