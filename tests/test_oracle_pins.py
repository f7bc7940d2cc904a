"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests compares the oracle with itself: each expected value is a
closed form, an invariant stated by an equation of the paper, a hand-computed
case, a brute-force evaluation in numpy written in a different form, or a
library eigensolver.
"""
import math

import numpy as np
import pytest

from paper_1811_03617_b200 import workloads as W


def _np(t):
    return t.detach().cpu().numpy()


def _orthonormal(rng, d, k):
    q, _ = np.linalg.qr(rng.standard_normal((d, k)))
    return q


def _coarse(rng, shape, scale=1.0):
    """fp32 values on a 2^-8 grid with small magnitude: sums of a few of them are exact in fp32."""
    return (np.round(rng.standard_normal(shape) * 64 * scale) / 256.0).astype(np.float32)


# ------------------------------------------------------------------ P1: Eq. 1 / Eq. 4 linearity
def test_P1_sum_of_compressed_equals_compressed_sum(oracle):
    rng = np.random.default_rng(1)
    w = W.custom("p1", 101, d=16, k=4, N=5, L=1, layer_len=[16 * 37, 16 * 5 + 7, 16 * 11])
    g = [_coarse(rng, w.M) for _ in range(w.N)]
    Ut = np.stack([_orthonormal(rng, w.d, w.k).T for _ in range(w.n_layers)]).astype(np.float32)
    mu = _coarse(rng, (w.n_layers, w.d))
    s_sum = oracle.aggregate([oracle.compress(w, gn, Ut, mu, w.N) for gn in g])
    # right-hand side of Eq. 4, written as one matrix product per layer in numpy
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    rows = []
    for l in range(w.n_layers):
        S = w.layer_len[l] // w.d
        X = gsum[w.layer_off[l]: w.layer_off[l] + S * w.d].reshape(S, w.d)
        rows.append((X - mu[l].astype(np.float64)) @ Ut[l].astype(np.float64).T)
    rhs = np.concatenate(rows)
    assert s_sum.shape == rhs.shape
    assert np.linalg.norm(s_sum - rhs) <= 1e-12 * np.linalg.norm(rhs)


def test_P1_two_node_additivity(oracle):
    # Q(g1) + Q(g2) = U^T (g1 + g2 - 2 mu / N): the compressor is affine with offset mu / N per node
    rng = np.random.default_rng(2)
    w = W.custom("p1b", 102, d=8, k=3, N=4, L=1, layer_len=[8 * 50])
    g1, g2 = _coarse(rng, w.M), _coarse(rng, w.M)
    Ut = _orthonormal(rng, 8, 3).T[None].astype(np.float32)
    mu = _coarse(rng, (1, 8))
    lhs = oracle.compress(w, g1, Ut, mu, 4) + oracle.compress(w, g2, Ut, mu, 4)
    X = (g1.astype(np.float64) + g2.astype(np.float64)).reshape(-1, 8) - 2.0 * mu[0].astype(np.float64) / 4.0
    rhs = X @ Ut[0].astype(np.float64).T
    assert np.linalg.norm(lhs - rhs) <= 1e-12 * np.linalg.norm(rhs)
    # and with N = 1 a node's own mean is removed entirely: compress(mu) = 0
    z = oracle.compress(w, np.tile(mu[0], 50), Ut, mu, 1)
    assert np.abs(z).max() == 0.0


def test_P1_compress_matches_hand_computed_case(oracle):
    # d = 4, k = 2, N = 2; Ut rows e0 and (e1 + e2) / sqrt(2) rounded to fp32; mu = (2, 4, 6, 8)
    w = W.custom("hand", 103, d=4, k=2, N=2, L=1, layer_len=[8])
    r = np.float32(math.sqrt(0.5))
    Ut = np.array([[[1, 0, 0, 0], [0, r, r, 0]]], dtype=np.float32)
    mu = np.array([[2, 4, 6, 8]], dtype=np.float32)
    g = np.array([1, 2, 3, 4, 5, 6, 7, 8], dtype=np.float32)
    s = oracle.compress(w, g, Ut, mu, 2)
    # slice 0: x - mu/2 = (0, 0, 0, 0);  slice 1: (4, 4, 4, 4)
    expect = np.array([[0.0, 0.0], [4.0, 8.0 * float(r)]])
    assert np.allclose(s, expect, rtol=0, atol=1e-15)


# ------------------------------------------------------------------ P3: k = d is lossless
@pytest.mark.parametrize("d", [4, 16, 32])
def test_P3_full_rank_roundtrip_returns_the_sum(oracle, d):
    rng = np.random.default_rng(3 + d)
    w = W.custom("p3", 104, d=d, k=d, N=3, L=1, layer_len=[d * 21, d * 2 + d // 2])
    g = [rng.standard_normal(w.M).astype(np.float32) for _ in range(3)]
    Ut = np.stack([_orthonormal(rng, d, d).T for _ in range(2)]).astype(np.float32)
    mu = rng.standard_normal((2, d)).astype(np.float32)
    s_sum, g_hat = oracle.pipeline(w, g, Ut, mu)
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    # Ut is orthogonal only to fp32 rounding (1e-7), so that is the achievable accuracy
    assert np.linalg.norm(g_hat - gsum) <= 5e-6 * np.linalg.norm(gsum)
    # with an exactly orthogonal basis (a signed permutation) the round trip is exact to 1e-15
    P = np.zeros((2, d, d), dtype=np.float32)
    for l in range(2):
        perm = rng.permutation(d)
        P[l, np.arange(d), perm] = rng.choice([-1.0, 1.0], d)
    _, g_hat = oracle.pipeline(w, g, P, mu)
    assert np.linalg.norm(g_hat - gsum) <= 1e-14 * np.linalg.norm(gsum)


# ------------------------------------------------------------------ P8: tails and short layers are plain sums
def test_P8_tail_and_short_layers_are_plain_sums(oracle):
    rng = np.random.default_rng(8)
    w = W.custom("p8", 105, d=16, k=4, N=6, L=1, layer_len=[5, 16 * 3 + 15, 12, 16])
    g = [rng.standard_normal(w.M).astype(np.float32) for _ in range(w.N)]
    Ut = np.stack([_orthonormal(rng, 16, 4).T for _ in range(4)]).astype(np.float32)
    mu = rng.standard_normal((4, 16)).astype(np.float32)
    s_sum, g_hat = oracle.pipeline(w, g, Ut, mu)
    assert s_sum.shape == (4, 4)  # 0 + 3 + 0 + 1 slices
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    for l, (off, m) in enumerate(zip(w.layer_off, w.layer_len)):
        S = m // 16
        tail = slice(off + S * 16, off + m)
        assert np.array_equal(g_hat[tail], gsum[tail])
    # compressed part differs from the plain sum (k < d), so tails were not produced by Eq. 5
    assert np.linalg.norm(g_hat[5:5 + 48] - gsum[5:5 + 48]) > 1e-3


# ------------------------------------------------------------------ P5: the eigen routine
def test_P5_jacobi_2x2_closed_form(oracle):
    a, b, c = 2.0, -1.5, 0.25
    diag, V, _ = oracle.jacobi_eig(np.array([[a, b], [b, c]]))
    disc = math.sqrt((a - c) ** 2 / 4 + b * b)
    expect = sorted([(a + c) / 2 + disc, (a + c) / 2 - disc])
    assert np.allclose(sorted(diag), expect, rtol=1e-14)


def test_P5_jacobi_diagonal_and_zero(oracle):
    diag, V, sweeps = oracle.jacobi_eig(np.diag([3.0, -1.0, 7.0, 0.0]))
    assert sweeps == 0 and np.array_equal(diag, [3.0, -1.0, 7.0, 0.0]) and np.array_equal(V, np.eye(4))
    diag, V, _ = oracle.jacobi_eig(np.zeros((5, 5)))
    assert np.array_equal(diag, np.zeros(5)) and np.array_equal(V, np.eye(5))


@pytest.mark.parametrize("n", [3, 8, 33, 64])
def test_P5_jacobi_recovers_constructed_spectrum(oracle, n):
    rng = np.random.default_rng(50 + n)
    lam = np.sort(rng.uniform(0.1, 10.0, n))[::-1].copy()
    lam[-1] = 0.0  # a singular PSD matrix
    Q = np.eye(n)
    for _ in range(3):  # product of Householder reflectors
        v = rng.standard_normal(n)
        v /= np.linalg.norm(v)
        Q = Q @ (np.eye(n) - 2.0 * np.outer(v, v))
    C = (Q * lam) @ Q.T
    C = (C + C.T) / 2
    diag, V, _ = oracle.jacobi_eig(C)
    order = np.argsort(-diag)
    assert np.allclose(diag[order], lam, atol=1e-12 * lam[0])
    assert np.abs(V.T @ V - np.eye(n)).max() <= 1e-12
    assert np.linalg.norm(C @ V - V * diag) <= 1e-12 * np.linalg.norm(C)
    # eigenvectors agree with the construction up to sign (the spectrum is simple)
    assert np.allclose(np.abs(V[:, order].T @ Q), np.eye(n), atol=1e-9)


def test_P5_jacobi_agrees_with_library_eigh(oracle):
    rng = np.random.default_rng(55)
    X = rng.standard_normal((200, 48))
    C = X.T @ X / 200
    diag, V, _ = oracle.jacobi_eig(C)
    lib = np.linalg.eigh(C)[0][::-1]
    assert np.allclose(np.sort(diag)[::-1], lib, rtol=1e-12)


def test_P5_sort_order_and_sign(oracle):
    # eigenvalues (1, 5, 5, 3): the two equal ones keep their original order (index 1 before 2)
    V = np.eye(4)[:, [0, 1, 2, 3]].copy()
    V[:, 1] = [0.0, -1.0, 0.0, 0.0]  # largest-magnitude entry negative: must be flipped
    V[:, 2] = [0.0, 0.0, 0.6, -0.8]  # largest magnitude is the negative one: flipped
    ev, Ut = oracle.sort_eigs(np.array([1.0, 5.0, 5.0, 3.0]), V, 3)
    assert np.array_equal(ev, [5.0, 5.0, 3.0, 1.0])
    assert np.array_equal(Ut[0], [0.0, 1.0, 0.0, 0.0])
    assert np.allclose(Ut[1], [0.0, 0.0, -0.6, 0.8])
    assert np.array_equal(Ut[2], [0.0, 0.0, 0.0, 1.0])


# ------------------------------------------------------------------ P2 / P4 / P6: the fit
def _fit_tiny(oracle):
    w = W.tiny()
    hist = _np(W.stored_gradients(w))
    Ut, mu, ev, sw = oracle.fit_basis(w, hist, N=w.N, samples_are_sums_of=w.N)
    return w, hist, Ut, mu, ev


def test_P2_basis_is_orthonormal(oracle):
    w, hist, Ut, mu, ev = _fit_tiny(oracle)
    G = Ut[0] @ Ut[0].T
    assert np.abs(G - np.eye(w.k)).max() <= 1e-12
    G32 = Ut[0].astype(np.float32).astype(np.float64)
    assert np.abs(G32 @ G32.T - np.eye(w.k)).max() <= 1e-6
    assert np.all(np.diff(ev[0]) <= 0) and ev[0, -1] >= -1e-12


def test_P4_mean_cov_match_numpy_and_trace(oracle):
    w, hist, Ut, mu, ev = _fit_tiny(oracle)
    X = hist.reshape(-1, w.d).astype(np.float64)  # one layer, no tail: the samples are the rows
    assert np.allclose(mu[0], X.mean(axis=0), rtol=1e-13, atol=1e-13)
    C = np.cov(X.T, bias=True)  # 1/n normalisation
    assert np.isclose(ev[0].sum(), np.trace(C), rtol=1e-12)
    assert np.allclose(ev[0], np.linalg.eigvalsh(C)[::-1], rtol=1e-10, atol=1e-12 * ev[0, 0])


@pytest.mark.parametrize("k", [1, 4, 9, 16])
def test_P4_fit_set_residual_equals_discarded_eigenvalue_mass(oracle, k):
    # Eq. 6: the eigenvalue mass kept by the first k eigenvectors bounds the loss on the sample
    # slices; with the 1/n covariance the mean squared residual EQUALS the discarded mass.
    w = W.tiny()
    hist = _np(W.stored_gradients(w))
    Ut, mu, ev, _ = oracle.fit_basis(w, hist, N=1, samples_are_sums_of=1, k=k)
    X = hist.reshape(-1, w.d).astype(np.float64)
    Xc = X - mu[0]
    R = Xc - (Xc @ Ut[0].T) @ Ut[0]
    msr = (R ** 2).sum() / X.shape[0]
    assert np.isclose(msr, ev[0, k:].sum(), rtol=1e-9, atol=1e-12 * ev[0].sum())
    # the same through the oracle's own Eq. 3 / Eq. 5 / Eq. 7 on the fp32-rounded basis
    Ut32, mu32 = Ut.astype(np.float32), mu.astype(np.float32)
    total = 0.0
    for h in range(hist.shape[0]):
        total += oracle.local_loss(w, hist[h], Ut32, mu32, 1, k=k)
        s = oracle.compress(w, hist[h], Ut32, mu32, 1, k=k)
        g_hat = oracle.decompress(w, s, Ut32, mu32, None, 1, w.M, k=k)
        assert np.isclose(((g_hat - hist[h]) ** 2).sum(), oracle.local_loss(w, hist[h], Ut32, mu32, 1, k=k),
                          rtol=1e-9, atol=1e-9)
    tol = 1e-5 * ev[0].sum()
    assert abs(total / X.shape[0] - ev[0, k:].sum()) <= tol


def test_P4_aggregate_mean_convention(oracle):
    # samples that are sums of c nodes: mu = (N / c) * sample mean
    w = W.tiny()
    hist = _np(W.stored_gradients(w, L=2))
    m = hist.reshape(-1, w.d).astype(np.float64).mean(axis=0)
    for N, c in ((4, 4), (4, 1), (6, 3)):
        _, mu, _, _ = oracle.fit_basis(w, hist, N=N, samples_are_sums_of=c)
        assert np.allclose(mu[0], m * N / c, rtol=1e-13)


def test_P6_projector_idempotent_and_subspace_reproduced(oracle):
    rng = np.random.default_rng(6)
    w = W.custom("p6", 106, d=16, k=4, N=1, L=1, layer_len=[16 * 40])
    # an exactly orthonormal fp32 basis: normalised Hadamard columns (entries +-0.25)
    H = np.array([[1]])
    for _ in range(4):
        H = np.block([[H, H], [H, -H]])
    Ut = (H[:4] / 4.0).astype(np.float32)[None]
    mu = _coarse(rng, (1, 16))
    c = _coarse(rng, (40, 4))
    X = (c.astype(np.float64) @ Ut[0].astype(np.float64) + mu[0]).astype(np.float32)  # exact in fp32
    s = oracle.compress(w, X.reshape(-1), Ut, mu, 1)
    assert np.allclose(s, c, atol=1e-13)
    g_hat = oracle.decompress(w, s, Ut, mu, None, 1, w.M)
    assert np.allclose(g_hat, X.reshape(-1), atol=1e-13)
    # idempotence on arbitrary input: compress(decompress(compress(x))) = compress(x)
    Y = rng.standard_normal(w.M).astype(np.float32)
    s1 = oracle.compress(w, Y, Ut, mu, 1)
    y1 = oracle.decompress(w, s1, Ut, mu, None, 1, w.M)
    # y1 is float64; feed its fp32 rounding back
    s2 = oracle.compress(w, y1.astype(np.float32), Ut, mu, 1)
    assert np.linalg.norm(s2 - s1) <= 1e-6 * np.linalg.norm(s1)


def test_P7_fit_recovers_the_planted_subspace(oracle):
    # x = mu + A z + eps with tiny eps: span(U) -> span(A), and k eigenvalues carry the mass
    w = W.tiny()  # sigma = 0.01 absolute
    hist = _np(W.stored_gradients(w))
    Ut, mu, ev, _ = oracle.fit_basis(w, hist, N=w.N, samples_are_sums_of=w.N)
    _, A, sigma = W.layer_params(w, 0)
    Qa, _ = np.linalg.qr(_np(A).astype(np.float64))
    sv = np.linalg.svd(Ut[0] @ Qa, compute_uv=False)
    angle = math.acos(min(1.0, sv.min()))
    assert angle < 5e-3
    # noise eigenvalues of a sum of N node draws: N sigma^2 each
    assert np.allclose(ev[0, w.k:], w.N * sigma ** 2, rtol=0.2)
    assert ev[0, w.k - 1] > 1e3 * ev[0, w.k]
    # planted mean: N * mu_l
    m, _, _ = W.layer_params(w, 0)
    assert np.abs(mu[0] - w.N * _np(m)).max() < 0.3


def test_fit_many_layers_matches_per_layer_numpy(oracle):
    w = W.custom("fitm", 107, d=8, k=2, N=2, L=3, layer_len=[8 * 30 + 3, 5, 8 * 12], literal_sums=True)
    hist = _np(W.stored_gradients(w))
    Ut, mu, ev, sw = oracle.fit_basis(w, hist, N=2, samples_are_sums_of=2)
    for l in (0, 2):
        S = w.layer_len[l] // 8
        X = hist[:, w.layer_off[l]: w.layer_off[l] + S * 8].reshape(-1, 8).astype(np.float64)
        lam, vec = np.linalg.eigh(np.cov(X.T, bias=True))
        assert np.allclose(ev[l], lam[::-1], rtol=1e-10, atol=1e-13)
        P_lib = vec[:, -2:] @ vec[:, -2:].T
        assert np.allclose(Ut[l].T @ Ut[l], P_lib, atol=1e-9)
        assert np.allclose(mu[l], X.mean(axis=0), rtol=1e-13)
    # a layer with no full slice gets an orthonormal placeholder and zero eigenvalues
    assert np.array_equal(ev[1], np.zeros(8)) and np.array_equal(Ut[1], np.eye(8)[:2])


# ------------------------------------------------------------------ P10: Eq. 6
def test_P14_fit_from_summed_moments_equals_the_direct_fit(oracle):
    """Covariance and mean do not depend on the point the moments are taken about, and moments add over any split
    of the samples: the fit assembled from two participants' moments about an arbitrary common centre is the fit
    of all samples at once."""
    rng = np.random.default_rng(14)
    w = W.custom("p14", 114, d=12, k=3, N=4, L=6, layer_len=[12 * 40 + 5, 7, 12 * 9])
    hist = (rng.standard_normal((w.L, w.M)) * 0.5 + 3.0).astype(np.float32)
    hist[:, : 12 * 40] += np.tile(np.linspace(-2, 2, 12), 40).astype(np.float32)
    Ut_d, mu_d, ev_d, _ = oracle.fit_basis(w, hist, N=w.N, samples_are_sums_of=w.N)
    for centre in (np.zeros((3, 12)), rng.standard_normal((3, 12)) + 3.0):
        parts = [oracle.fit_moments(w, hist[:2], centre), oracle.fit_moments(w, hist[2:], centre)]
        assert parts[0][0, 0] == 2 * 40 and parts[1][0, 0] == 4 * 40 and parts[0][1, 0] == 0
        Ut_m, mu_m, ev_m = oracle.fit_from_moments(w, parts[0] + parts[1], centre, w.N, w.N)
        assert np.abs(ev_m - ev_d).max() <= 1e-10 * ev_d.max()
        assert np.abs(mu_m - mu_d).max() <= 1e-10 * np.abs(mu_d).max()
        for l in (0, 2):
            P = Ut_m[l] - (Ut_m[l] @ Ut_d[l].T) @ Ut_d[l]
            assert np.linalg.norm(P, 2) <= 1e-8
        assert np.array_equal(Ut_m[1], np.eye(12)[:3]) and np.all(ev_m[1] == 0)     # a layer without a full slice
    # the moments themselves against numpy on one layer
    X = hist[:, : 12 * 40].reshape(-1, 12).astype(np.float64)
    m = oracle.fit_moments(w, hist, np.zeros((3, 12)))[0]
    assert np.allclose(m[1:13], X.sum(0), rtol=1e-13) and np.allclose(m[13:].reshape(12, 12), X.T @ X, rtol=1e-13)
    assert np.allclose(np.cov(X.T, bias=True), m[13:].reshape(12, 12) / m[0] - np.outer(m[1:13], m[1:13]) / m[0] ** 2,
                       rtol=1e-9, atol=1e-12)


def test_P10_select_k(oracle):
    assert oracle.select_k(np.ones(4), 0.25) == 3          # 3/4 >= 0.75, inclusive
    assert oracle.select_k(np.ones(4), 0.2499) == 4
    assert oracle.select_k(np.ones(4), 0.0) == 4
    assert oracle.select_k(np.array([8.0, 4.0, 2.0, 1.0, 1.0]), 0.5) == 1  # 8/16
    assert oracle.select_k(np.array([8.0, 4.0, 2.0, 1.0, 1.0]), 0.25) == 2  # 12/16
    assert oracle.select_k(np.array([8.0, 4.0, 2.0, 1.0, 1.0]), 0.24) == 3
    assert oracle.select_k(np.zeros(6), 0.01) == 0          # degenerate spectrum
    # the synthetic workloads carry (almost) all mass in k directions
    lam = np.array([100.0] * 8 + [0.01] * 56)
    assert oracle.select_k(lam, 0.01) == 8


# ------------------------------------------------------------------ P9: the quantizer
def _py_mix(z):
    M = (1 << 64) - 1
    z ^= z >> 30; z = (z * 0xBF58476D1CE4E5B9) & M
    z ^= z >> 27; z = (z * 0x94D049BB133111EB) & M
    z ^= z >> 31
    return z


def _py_hash24(seed, node, sl, coord):
    M, M32 = (1 << 64) - 1, (1 << 32) - 1
    h = _py_mix((seed + 0x9E3779B97F4A7C15 * (node + 1)) & M)
    h = _py_mix(h ^ ((0xD1B54A32D192ED03 * (sl + 1)) & M))
    x = (h >> 32) ^ (((h & M32) + 0x9E3779B9 * (coord + 1)) & M32)
    x ^= x >> 16; x = (x * 0x7FEB352D) & M32
    x ^= x >> 15; x = (x * 0x846CA68B) & M32
    x ^= x >> 16
    return x >> 8


def test_P9_hash_is_the_documented_mixer(oracle):
    for key in [(0, 0, 0, 0), (1, 2, 3, 4), (2 ** 64 - 1, 2 ** 32 - 1, 2 ** 40 + 12345, 255), (20181103, 31, 390143, 31)]:
        assert oracle.hash24(*key) == _py_hash24(*key)


def test_P9_hash_uniform_and_key_sensitive(oracle):
    h = np.array([oracle.hash24(7, n, s, c) for n in range(4) for s in range(64) for c in range(32)], dtype=np.float64)
    u = h / 2 ** 24
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / u.size)
    counts = np.histogram(u, bins=16, range=(0, 1))[0]
    chi2 = ((counts - u.size / 16) ** 2 / (u.size / 16)).sum()
    assert chi2 < 45  # 15 dof, p ~ 1e-4
    # adjacent coordinates / slices / nodes are uncorrelated (lag-1 correlation of each key direction)
    g = u.reshape(4, 64, 32) - 0.5
    for a, b in ((g[:, :, 1:], g[:, :, :-1]), (g[:, 1:, :], g[:, :-1, :]), (g[1:], g[:-1])):
        r = (a * b).mean() * 12
        assert abs(r) < 5 / math.sqrt(a.size)
    base = oracle.hash24(7, 1, 2, 3)
    assert len({base, oracle.hash24(8, 1, 2, 3), oracle.hash24(7, 2, 2, 3), oracle.hash24(7, 1, 3, 3),
                oracle.hash24(7, 1, 2, 4)}) == 5


def test_P9_exact_when_ratios_are_integers(oracle):
    v = np.array([[3.0, -4.0, 0.0, 0.0], [0.0, 0.0, 0.0, 0.0], [-0.0, 5.0, 0.0, 12.0]], dtype=np.float32)
    for seed in range(5):
        q, norms = oracle.quantize(v, 5 if seed < 3 else 65, seed, node=seed)
        lv = 5 if seed < 3 else 65
        assert np.array_equal(norms, np.array([5.0, 0.0, 13.0], dtype=np.float32))
        assert np.array_equal(q[0], np.array([3, -4, 0, 0]) * (lv // 5))
        assert np.array_equal(q[1], [0, 0, 0, 0])
        if lv == 65:
            assert np.array_equal(q[2], [0, 25, 0, 60])


def test_P9_norm_uses_the_butterfly_order(oracle):
    # squares (2^-24, 2^-24, 1, 0): butterfly = (a0 + a2) + (a1 + a3) = fl(1 + 2^-24) + 2^-24 -> 1 -> 1
    # (a left-to-right sum would give 1 + 2^-23)
    v = np.array([[2.0 ** -12, 2.0 ** -12, 1.0, 0.0]], dtype=np.float32)
    _, norms = oracle.quantize(v, 7, 0, 0)
    assert norms[0] == np.float32(1.0)
    # k = 3 pads one zero: (a0 + a2) + (a1 + 0)
    v = np.array([[1.0, 2.0 ** -12, 2.0 ** -12]], dtype=np.float32)
    _, norms = oracle.quantize(v, 7, 0, 0)
    a = np.float32(1.0) + np.float32(2.0 ** -24)
    assert norms[0] == np.sqrt(np.float32(a + np.float32(2.0 ** -24)))


def test_P9_levels_bounded_adjacent_and_signed(oracle):
    rng = np.random.default_rng(9)
    v = rng.standard_normal((500, 32)).astype(np.float32)
    v[3] = 0.0
    v[4, 1:] = 0.0  # a single non-zero coordinate: ratio = levels exactly
    for levels in (1, 7, 127):
        q, norms = oracle.quantize(v, levels, 99, 3, slice0=1000)
        assert q.min() >= -levels and q.max() <= levels
        nrm = np.sqrt((v.astype(np.float64) ** 2).sum(axis=1))
        assert np.allclose(norms, nrm, rtol=1e-6)
        r = levels * np.abs(v.astype(np.float64)) / np.where(nrm > 0, nrm, 1.0)[:, None]
        assert np.all(np.abs(np.abs(q) - r) < 1.0 + 1e-4)
        assert np.all((q == 0) | (np.sign(q) == np.sign(v)))
        assert np.array_equal(q[3], np.zeros(32)) and abs(q[4, 0]) == levels and np.all(q[4, 1:] == 0)


def test_P9_unbiased(oracle):
    # E[norm * q / levels] = v : average over many seeds converges like 1 / sqrt(trials)
    rng = np.random.default_rng(10)
    v = rng.standard_normal((8, 16)).astype(np.float32)
    levels, trials = 7, 4000
    acc = np.zeros(v.shape)
    for seed in range(trials):
        q, norms = oracle.quantize(v, levels, seed, node=1)
        acc += norms[:, None].astype(np.float64) * q / levels
    mean = acc / trials
    # per-coordinate std of one draw <= norm / (2 levels)
    bound = 5.0 * (np.linalg.norm(v, axis=1)[:, None] / (2 * levels)) / math.sqrt(trials)
    assert np.all(np.abs(mean - v) <= bound + 1e-6)
    # different nodes / slices draw different randomness
    q0, _ = oracle.quantize(v, levels, 5, node=0)
    q1, _ = oracle.quantize(v, levels, 5, node=1)
    q2, _ = oracle.quantize(v, levels, 5, node=0, slice0=8)
    assert np.any(q0 != q1) and np.any(q0 != q2)
    # slice0 shifts the counter: rows 4.. of a call at slice0=0 equal rows 0.. of a call at slice0=4
    qa, _ = oracle.quantize(v, levels, 5, node=0)
    qb, _ = oracle.quantize(v[4:], levels, 5, node=0, slice0=4)
    assert np.array_equal(qa[4:], qb)


def test_P9_dequantize_aggregate_is_the_weighted_sum(oracle):
    rng = np.random.default_rng(11)
    qs = [rng.integers(-7, 8, (20, 8)).astype(np.int8) for _ in range(3)]
    ns = [rng.uniform(0, 3, 20).astype(np.float32) for _ in range(3)]
    out = oracle.dequantize_aggregate(qs, ns, 7)
    expect = sum(n.astype(np.float64)[:, None] * q / 7.0 for q, n in zip(qs, ns))
    assert np.allclose(out, expect, rtol=1e-14, atol=1e-15)


def test_P9_quantized_pipeline_is_within_one_level_per_node_and_unbiased(oracle):
    """The path with the quantizer between Eq. 3 and Eq. 4: every node's dequantised vector is within norm / levels
    of its s_n per coordinate, so the aggregate is within sum_n norm_n / levels of the unquantized one, and averaged
    over seeds it converges to it (the quantizer is unbiased and Eq. 4 / Eq. 5 are linear)."""
    rng = np.random.default_rng(21)
    w = W.custom("p9pipe", 109, d=16, k=4, N=3, L=1, layer_len=[16 * 21, 16 * 6 + 5])
    g = [rng.standard_normal(w.M).astype(np.float32) for _ in range(w.N)]
    Ut = np.stack([_orthonormal(rng, w.d, w.k).T for _ in range(w.n_layers)]).astype(np.float32)
    mu = rng.standard_normal((w.n_layers, w.d)).astype(np.float32)
    levels = 7
    s_ref, g_ref = oracle.pipeline(w, g, Ut, mu)
    s_n = [oracle.compress(w, x, Ut, mu, w.N) for x in g]
    bound = sum(np.linalg.norm(s, axis=1) for s in s_n)[:, None] / levels
    acc_s, acc_g, trials = 0.0, 0.0, 600
    for seed in range(trials):
        s_q, g_q, qs, ns = oracle.pipeline_quantized(w, g, Ut, mu, levels, seed)
        assert np.all(np.abs(s_q - s_ref) <= bound * (1 + 1e-5) + 1e-6)
        assert all(q.dtype == np.int8 and np.abs(q).max() <= levels for q in qs)
        acc_s, acc_g = acc_s + s_q, acc_g + g_q
    # std of one draw of one coordinate <= sum_n norm_n / (2 levels); 5 sigma of the mean
    assert np.all(np.abs(acc_s / trials - s_ref) <= 5.0 * bound / 2 / math.sqrt(trials) + 1e-6)
    # the tails bypass the quantizer: identical in both paths
    ta = w.layer_off[1] + 16 * 6
    assert np.array_equal(g_q[ta:ta + 5], g_ref[ta:ta + 5])
    # Eq. 5 is linear: the mean reconstruction converges with the mean aggregate
    assert np.linalg.norm(acc_g / trials - g_ref) <= 0.05 * np.linalg.norm(g_ref)


def test_P11_flatten_order_matches_the_figure(oracle):
    """Section 2, figure on flattening and slicing: the worked 2 x 2 x 2 x 2 layer written out by hand in
    tests/golden/flatten_order.txt (digits f d h w), plus what any such order must satisfy."""
    from pathlib import Path
    want = [ln for ln in (Path(__file__).parent / "golden" / "flatten_order.txt").read_text().splitlines()
            if ln and not ln.startswith("#")][0].split()
    F = D = H = Wd = 2
    fw = np.zeros((F, D, H * Wd), dtype=np.float32)
    for f in range(F):
        for dd in range(D):
            for h in range(H):
                for w_ in range(Wd):
                    fw[f, dd, h * Wd + w_] = 1000 * f + 100 * dd + 10 * h + w_
    flat = oracle.flatten(fw).ravel()
    assert [f"{int(v):04d}" for v in flat] == want
    # a permutation with an inverse; every run of F entries shares its position; a slice of F * D entries holds
    # every filter and depth of one spatial position (what the paper slices by)
    rng = np.random.default_rng(12)
    F, D, X = 5, 3, 7
    fw = rng.standard_normal((F, D, X)).astype(np.float32)
    flat = oracle.flatten(fw)
    assert flat.shape == (X, D, F) and sorted(flat.ravel().tolist()) == sorted(fw.ravel().tolist())
    assert np.array_equal(oracle.flatten(flat, inverse=True), fw)
    for x in range(X):
        assert np.array_equal(flat[x], fw[:, :, x].T)


def test_P12_pack4_bytes_and_roundtrip(oracle):
    """Nibble packing: bytes worked out by hand (two's complement, even coordinate low), every level, round trip."""
    q = np.array([[0, 1, -1, 7, -7, 3, 2, -8 + 1]], dtype=np.int8)   # last = -7
    assert oracle.pack4(q).tolist() == [[0x10, 0x7F, 0x39, 0x92]]
    allq = np.array([[a, b] for a in range(-7, 8) for b in range(-7, 8)], dtype=np.int8)
    packed = oracle.pack4(allq)
    assert packed.shape == (225, 1) and len(set(packed.ravel().tolist())) == 225
    assert np.array_equal(oracle.unpack4(packed), allq)
    with pytest.raises(Exception):
        oracle.pack4(np.array([[8, 0]], dtype=np.int8))


def test_P12_quantize_raw4_is_the_bucket_quantizer_on_slices(oracle):
    """Raw-gradient quantization = the pinned bucket quantizer with bucket = slice, global slice index as counter,
    then packed; tails untouched; the aggregate is unbiased like the quantizer itself."""
    w = W.custom("raw4", 3, d=16, k=4, N=3, L=1, layer_len=[16 * 5 + 3, 7, 16 * 2])
    g = [t.numpy() for t in W.node_gradients(w)]
    q4, nrm = oracle.quantize_raw4(w, g[1], 7, 99, 1)
    assert q4.shape == (7, 8) and nrm.shape == (7,)
    q_l0, n_l0 = oracle.quantize(g[1][:80].reshape(5, 16), 7, 99, 1, slice0=0)
    q_l2, n_l2 = oracle.quantize(g[1][w.layer_off[2]:w.layer_off[2] + 32].reshape(2, 16), 7, 99, 1, slice0=5)
    assert np.array_equal(oracle.unpack4(q4), np.concatenate([q_l0, q_l2]))
    assert np.array_equal(nrm, np.concatenate([n_l0, n_l2]))
    outs = []
    for seed in range(300):
        qs = [oracle.quantize_raw4(w, x, 7, seed, n) for n, x in enumerate(g)]
        outs.append(oracle.dequantize_raw4_aggregate(w, [a for a, _ in qs], [b for _, b in qs], g, 7, w.M))
    mean = np.mean(outs, axis=0)
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    cov = ~np.isnan(mean)
    assert cov.sum() == sum(w.layer_len)
    tails = np.zeros(w.M, dtype=bool)
    for o, m in zip(w.layer_off, w.layer_len):
        tails[o + (m // 16) * 16:o + m] = True
    assert np.allclose(mean[tails], gsum[tails], rtol=1e-12)           # tails: plain sums
    nb = np.abs(mean[cov & ~tails] - gsum[cov & ~tails])
    assert nb.max() < 6.0 * np.abs(np.stack(g)).max() * 4 / 7 / np.sqrt(300)


# ------------------------------------------------------------------ P13: Algorithm 1 (ring schedule)
def _direct_result(w, g, Ut, mu):
    """Eq. 4's right-hand side put into Eq. 5, per layer in numpy: g_hat = (sum_n g_n - mu) U U^T + mu; tails summed."""
    gsum = np.sum(np.stack(g).astype(np.float64), axis=0)
    out = np.zeros(w.M)
    for l, (o, m) in enumerate(zip(w.layer_off, w.layer_len)):
        Sl = m // w.d
        X = gsum[o:o + Sl * w.d].reshape(Sl, w.d)
        U = Ut[l].astype(np.float64)
        out[o:o + Sl * w.d] = ((X - mu[l]) @ U.T @ U + mu[l]).reshape(-1)
        out[o + Sl * w.d:o + m] = gsum[o + Sl * w.d:o + m]
    return out


@pytest.mark.parametrize("N", [1, 2, 3, 4, 7])
def test_P13_segments_partition_the_slices_evenly(oracle, N):
    w = W.custom("p13a", 131, d=16, k=4, N=N, L=1, layer_len=[16 * 7 + 5, 9, 16 * 30, 16 * 3 + 2, 16 * 11, 3])
    segs = [oracle.segment_layout(w, N, j) for j in range(N)]
    covered = np.zeros(w.M, dtype=np.int32)
    for j, sg in enumerate(segs):
        assert (sg.slice0, sg.slice1) == ((j * w.S) // N, ((j + 1) * w.S) // N)
        assert sum(m // w.d for m in sg.layer_len) == sg.slice1 - sg.slice0
        for o, m in zip(sg.layer_off, sg.layer_len):
            covered[o:o + m] += 1
    counts = [sg.slice1 - sg.slice0 for sg in segs]
    assert max(counts) - min(counts) <= 1 and sum(counts) == w.S
    expect = np.zeros(w.M, dtype=np.int32)
    for o, m in zip(w.layer_off, w.layer_len):
        expect[o:o + m] = 1
    assert np.array_equal(covered, expect)          # every entry of every layer in exactly one segment


@pytest.mark.parametrize("N", [1, 2, 3, 5])
def test_P13_ring_gives_every_node_the_direct_result(oracle, N):
    rng = np.random.default_rng(13 + N)
    w = W.custom("p13b", 132, d=16, k=4, N=N, L=1, layer_len=[16 * 7 + 5, 9, 16 * 30, 16 * 3 + 2, 0, 16 * 11])
    g = [rng.standard_normal(w.M).astype(np.float32) for _ in range(N)]
    Ut = np.stack([_orthonormal(rng, w.d, w.k).T for _ in range(w.n_layers)]).astype(np.float32)
    mu = rng.standard_normal((w.n_layers, w.d)).astype(np.float32)
    expect = _direct_result(w, g, Ut, mu)
    g_hat, sent = oracle.ring_allreduce(w, g, Ut, mu)
    assert len(g_hat) == N
    for n in range(N):
        assert np.abs(g_hat[n] - expect).max() <= 1e-12 * max(1.0, np.abs(expect).max())
    # every segment crosses N - 1 links in each of the two rounds
    assert sum(sent) == 2 * (N - 1) * (w.S * w.k + w.tail_entries)
    if N > 1:
        assert max(sent) - min(sent) <= 2 * (N - 1) * (w.k + w.d)      # equal segments: equal load per link


def test_P13_without_compression_the_ring_is_a_plain_all_reduce(oracle):
    """k = d, U = I, mu = 0: Algorithm 1 with compression and decompression skipped is the ring all-reduce."""
    rng = np.random.default_rng(1313)
    N = 4
    w = W.custom("p13c", 133, d=8, k=8, N=N, L=1, layer_len=[8 * 9 + 3, 8 * 14])
    g = [_coarse(rng, w.M) for _ in range(N)]
    Ut = np.stack([np.eye(8, dtype=np.float32)] * w.n_layers)
    mu = np.zeros((w.n_layers, 8), dtype=np.float32)
    g_hat, sent = oracle.ring_allreduce(w, g, Ut, mu)
    total = np.sum(np.stack(g).astype(np.float64), axis=0)
    for n in range(N):
        assert np.array_equal(g_hat[n], total)     # coarse-grid inputs: the sums are exact
    assert sum(sent) == 2 * (N - 1) * w.M
