"""GradiVeQ oracle -- TEST INFRASTRUCTURE, not the product.

numpy/ctypes front end of ``gvq_oracle.c``: a plain fp64 CPU statement of the
GradiVeQ hot path (Eq. 3 compress, Eq. 4 aggregate, Eq. 5 decompress, the PCA
fit of Section 2, Eq. 6 / Eq. 7 helpers, the stochastic scalar quantizer, and
Algorithm 1's ring schedule simulated for N nodes in one process).
It shares nothing with the CUDA library and must only be used by the tests, the
smoke check and the benchmark's CPU-baseline / reference legs.

Arrays are numpy, C-contiguous.  ``layout`` is any object with integer
attributes ``d``, ``k`` and sequences ``layer_off``, ``layer_len``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "gvq_oracle.c"
_LIB = _HERE / "libgvq_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the C oracle with gcc (strict fp: no contraction, no fast-math)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-fPIC",
               "-shared", "-Wall", "-Wextra", str(_SRC), "-o", str(tmp), "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        lib.gvqo_local_loss.restype = ctypes.c_double
        lib.gvqo_hash24.restype = ctypes.c_uint32
        lib.gvqo_total_slices.restype = ctypes.c_int64
        _lib = lib
    return _lib


def _check(rc: int, what: str) -> None:
    if rc != 0:
        names = {1: "bad argument", 2: "Jacobi did not converge", 3: "out of memory"}
        raise RuntimeError(f"oracle {what}: {names.get(rc, rc)}")


def _p(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _i64(seq) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(seq, dtype=np.int64))


def _f32(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float32, a.dtype
    return a


def _layers(layout):
    off, ln = _i64(layout.layer_off), _i64(layout.layer_len)
    assert off.shape == ln.shape
    return off, ln


def total_slices(layout) -> int:
    return int(sum(int(m) // int(layout.d) for m in layout.layer_len))


def num_threads() -> int:
    """Threads the OpenMP loops of the oracle will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env:
        try:
            return max(1, int(env.split(",")[0]))
        except ValueError:
            pass
    return len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)


# --------------------------------------------------------------------------- eigen
def jacobi_eig(C: np.ndarray, max_sweeps: int = 100):
    """Eigenpairs of a symmetric matrix: returns (diag (unsorted), V (columns), sweeps)."""
    A = np.array(C, dtype=np.float64, order="C", copy=True)
    n = A.shape[0]
    assert A.shape == (n, n)
    V = np.empty((n, n), dtype=np.float64)
    sw = ctypes.c_int(0)
    rc = _load().gvqo_jacobi_eig(ctypes.c_int(n), _p(A, ctypes.c_double), _p(V, ctypes.c_double),
                                 ctypes.c_int(max_sweeps), ctypes.byref(sw))
    _check(rc, "jacobi_eig")
    return np.diag(A).copy(), V, sw.value


def sort_eigs(diag: np.ndarray, V: np.ndarray, k: int):
    """Descending eigenvalues and the first k eigenvectors as rows (sign-fixed)."""
    n = V.shape[0]
    A = np.ascontiguousarray(np.diag(np.asarray(diag, dtype=np.float64)))
    V = np.ascontiguousarray(V, dtype=np.float64)
    ev = np.empty(n, dtype=np.float64)
    Ut = np.empty((k, n), dtype=np.float64)
    rc = _load().gvqo_sort_eigs(ctypes.c_int(n), ctypes.c_int(k), _p(A, ctypes.c_double),
                                _p(V, ctypes.c_double), _p(ev, ctypes.c_double), _p(Ut, ctypes.c_double))
    _check(rc, "sort_eigs")
    return ev, Ut


def mean_cov(d: int, layer_off: int, layer_len: int, hist: np.ndarray):
    """Sample mean and 1/n covariance of one layer's slices over the L stored gradients."""
    hist = _f32(hist)
    assert hist.ndim == 2
    mean = np.empty(d, dtype=np.float64)
    cov = np.empty((d, d), dtype=np.float64)
    rc = _load().gvqo_mean_cov(ctypes.c_int(d), ctypes.c_int64(layer_off), ctypes.c_int64(layer_len),
                               _p(hist, ctypes.c_float), ctypes.c_int64(hist.shape[1]),
                               ctypes.c_int(hist.shape[0]), _p(mean, ctypes.c_double),
                               _p(cov, ctypes.c_double))
    _check(rc, "mean_cov")
    return mean, cov


def fit_basis(layout, hist: np.ndarray, N: int, samples_are_sums_of: int, k: int | None = None):
    """PCA fit per layer.  hist [L][M] fp32.  Returns (Ut [layers][k][d], mu [layers][d],
    evals [layers][d], sweeps [layers]) with Ut, mu, evals in float64."""
    hist = _f32(hist)
    assert hist.ndim == 2
    d = int(layout.d)
    k = int(layout.k if k is None else k)
    off, ln = _layers(layout)
    nl = len(off)
    Ut = np.zeros((nl, k, d), dtype=np.float64)
    mu = np.zeros((nl, d), dtype=np.float64)
    ev = np.zeros((nl, d), dtype=np.float64)
    sw = np.zeros(nl, dtype=np.int32)
    rc = _load().gvqo_fit_basis(ctypes.c_int(d), ctypes.c_int(k), ctypes.c_int(nl), _p(off, ctypes.c_int64),
                                _p(ln, ctypes.c_int64), _p(hist, ctypes.c_float),
                                ctypes.c_int64(hist.shape[1]), ctypes.c_int(hist.shape[0]), ctypes.c_int(N),
                                ctypes.c_int(samples_are_sums_of), _p(Ut, ctypes.c_double),
                                _p(mu, ctypes.c_double), _p(ev, ctypes.c_double), _p(sw, ctypes.c_int32))
    _check(rc, "fit_basis")
    return Ut, mu, ev, sw


def fit_moments(layout, hist: np.ndarray, centre: np.ndarray) -> np.ndarray:
    """Additive moments of the sample slices of `hist` [L][M] about `centre` [layers][d] (Section 2: the covariance
    of samples that are spread over several nodes is assembled from sums): per layer
    [n, sum (x - m), sum (x - m)(x - m)^T] in float64, shape [layers][1 + d + d * d]."""
    hist = _f32(hist)
    d = int(layout.d)
    off, ln = _layers(layout)
    out = np.zeros((len(off), 1 + d + d * d), dtype=np.float64)
    for l, (o, m) in enumerate(zip(off, ln)):
        S = int(m) // d
        if S == 0:
            continue
        X = hist[:, int(o):int(o) + S * d].reshape(-1, d).astype(np.float64) - np.asarray(centre[l], dtype=np.float64)
        out[l, 0] = X.shape[0]
        out[l, 1:1 + d] = X.sum(axis=0)
        out[l, 1 + d:] = (X.T @ X).ravel()
    return out


def fit_from_moments(layout, moments: np.ndarray, centre: np.ndarray, N: int, samples_are_sums_of: int,
                     k: int | None = None):
    """The PCA fit from summed moments: C = S2 / n - delta delta^T, mean = m + delta with delta = sum (x - m) / n,
    then the eigendecomposition, ordering and sign rule of fit_basis.  Returns (Ut, mu, evals) in float64."""
    d = int(layout.d)
    k = int(layout.k if k is None else k)
    nl = moments.shape[0]
    Ut = np.zeros((nl, k, d)); mu = np.zeros((nl, d)); ev = np.zeros((nl, d))
    for l in range(nl):
        n = moments[l, 0]
        if n <= 0:
            Ut[l] = np.eye(d)[:k]
            continue
        delta = moments[l, 1:1 + d] / n
        C = moments[l, 1 + d:].reshape(d, d) / n - np.outer(delta, delta)
        diag, V, _ = jacobi_eig(0.5 * (C + C.T))
        ev[l], Ut[l] = sort_eigs(diag, V, k)
        mu[l] = (np.asarray(centre[l], dtype=np.float64) + delta) * (float(N) / float(samples_are_sums_of))
    return Ut, mu, ev


# --------------------------------------------------------------------------- Eq. 3 / 4 / 5
def compress(layout, g_node: np.ndarray, Ut: np.ndarray, mu: np.ndarray, N: int, k: int | None = None):
    """Eq. 3 for one node: s [S_total][k] float64."""
    g_node, Ut, mu = _f32(g_node), _f32(Ut), _f32(mu)
    d = int(layout.d)
    k = int(layout.k if k is None else k)
    off, ln = _layers(layout)
    s = np.zeros((total_slices(layout), k), dtype=np.float64)
    rc = _load().gvqo_compress(ctypes.c_int(d), ctypes.c_int(k), ctypes.c_int(len(off)),
                               _p(off, ctypes.c_int64), _p(ln, ctypes.c_int64), _p(g_node, ctypes.c_float),
                               _p(Ut, ctypes.c_float), _p(mu, ctypes.c_float), ctypes.c_int(N),
                               _p(s, ctypes.c_double))
    _check(rc, "compress")
    return s


def aggregate(s_nodes):
    """Eq. 4: elementwise sum of the nodes' compressed buffers (float64)."""
    arrs = [np.ascontiguousarray(a, dtype=np.float64) for a in s_nodes]
    out = np.empty_like(arrs[0])
    ptrs = (ctypes.POINTER(ctypes.c_double) * len(arrs))(*[_p(a, ctypes.c_double) for a in arrs])
    rc = _load().gvqo_aggregate(ctypes.c_int64(out.size), ctypes.c_int(len(arrs)), ptrs,
                                _p(out, ctypes.c_double))
    _check(rc, "aggregate")
    return out


def decompress(layout, s_sum: np.ndarray, Ut: np.ndarray, mu: np.ndarray, g_nodes, N: int,
               M: int, k: int | None = None):
    """Eq. 5 plus the raw tails: flat g_hat of length M in float64 (gaps stay 0)."""
    Ut, mu = _f32(Ut), _f32(mu)
    s_sum = np.ascontiguousarray(s_sum, dtype=np.float64)
    d = int(layout.d)
    k = int(layout.k if k is None else k)
    off, ln = _layers(layout)
    g_hat = np.zeros(M, dtype=np.float64)
    if g_nodes is not None:
        gs = [_f32(g) for g in g_nodes]
        ptrs = (ctypes.POINTER(ctypes.c_float) * len(gs))(*[_p(g, ctypes.c_float) for g in gs])
    else:
        ptrs = None
    rc = _load().gvqo_decompress(ctypes.c_int(d), ctypes.c_int(k), ctypes.c_int(len(off)),
                                 _p(off, ctypes.c_int64), _p(ln, ctypes.c_int64), _p(s_sum, ctypes.c_double),
                                 _p(Ut, ctypes.c_float), _p(mu, ctypes.c_float), ptrs, ctypes.c_int(N),
                                 _p(g_hat, ctypes.c_double))
    _check(rc, "decompress")
    return g_hat


def select_k(evals: np.ndarray, lambda_loss: float) -> int:
    """Eq. 6: smallest k whose leading eigenvalue mass reaches 1 - lambda_loss (0 if the mass is 0)."""
    ev = np.ascontiguousarray(evals, dtype=np.float64)
    return int(_load().gvqo_select_k(ctypes.c_int(ev.size), _p(ev, ctypes.c_double),
                                     ctypes.c_double(lambda_loss)))


def local_loss(layout, g_node, Ut, mu, N: int, k: int | None = None) -> float:
    """Eq. 7: one node's squared reconstruction error over all its slices."""
    g_node, Ut, mu = _f32(g_node), _f32(Ut), _f32(mu)
    d = int(layout.d)
    k = int(layout.k if k is None else k)
    off, ln = _layers(layout)
    return float(_load().gvqo_local_loss(ctypes.c_int(d), ctypes.c_int(k), ctypes.c_int(len(off)),
                                         _p(off, ctypes.c_int64), _p(ln, ctypes.c_int64),
                                         _p(g_node, ctypes.c_float), _p(Ut, ctypes.c_float),
                                         _p(mu, ctypes.c_float), ctypes.c_int(N)))


def flatten(framework: np.ndarray, inverse: bool = False) -> np.ndarray:
    """The paper's flatten order of one layer.  framework: [F][D][X] (X = H * W, row-major) -> flat [X * D * F];
    inverse: flat [X][D][F] -> [F][D][X]."""
    a = _f32(framework)
    assert a.ndim == 3
    if inverse:
        X, D, F = a.shape
        out = np.zeros((F, D, X), dtype=np.float32)
    else:
        F, D, X = a.shape
        out = np.zeros((X, D, F), dtype=np.float32)
    _check(_load().gvqo_flatten(ctypes.c_int(F), ctypes.c_int(D), ctypes.c_int(X), _p(a, ctypes.c_float),
                                _p(out, ctypes.c_float), ctypes.c_int(1 if inverse else 0)), "flatten")
    return out


# --------------------------------------------------------------------------- quantizer
def hash24(seed: int, node: int, slice_index: int, coord: int) -> int:
    """The 24 random bits the quantizer draws for (seed, node, slice, coordinate)."""
    return int(_load().gvqo_hash24(ctypes.c_uint64(seed), ctypes.c_uint32(node), ctypes.c_uint64(slice_index),
                                   ctypes.c_uint32(coord)))


def quantize(s_node: np.ndarray, levels: int, seed: int, node: int, slice0: int = 0):
    """Stochastic scalar quantizer, one bucket per compressed slice: (q int8 [S][k], norms fp32 [S])."""
    s_node = _f32(s_node)
    assert s_node.ndim == 2
    S, k = s_node.shape
    q = np.zeros((S, k), dtype=np.int8)
    norms = np.zeros(S, dtype=np.float32)
    rc = _load().gvqo_quantize(ctypes.c_int(k), ctypes.c_int64(S), ctypes.c_int64(slice0),
                               _p(s_node, ctypes.c_float), ctypes.c_int(levels), ctypes.c_uint64(seed),
                               ctypes.c_uint32(node), _p(q, ctypes.c_int8), _p(norms, ctypes.c_float))
    _check(rc, "quantize")
    return q, norms


def pack4(q: np.ndarray) -> np.ndarray:
    """Signed levels in [-7, 7] -> two per byte (low nibble = even coordinate)."""
    q = np.ascontiguousarray(q, dtype=np.int8)
    out = np.zeros(q.size // 2, dtype=np.uint8)
    _check(_load().gvqo_pack4(ctypes.c_int64(q.size), _p(q, ctypes.c_int8), _p(out, ctypes.c_uint8)), "pack4")
    return out.reshape(q.shape[:-1] + (q.shape[-1] // 2,))


def unpack4(packed: np.ndarray) -> np.ndarray:
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    out = np.zeros(packed.size * 2, dtype=np.int8)
    _check(_load().gvqo_unpack4(ctypes.c_int64(out.size), _p(packed, ctypes.c_uint8), _p(out, ctypes.c_int8)), "unpack4")
    return out.reshape(packed.shape[:-1] + (packed.shape[-1] * 2,))


def quantize_raw4(layout, g_node: np.ndarray, levels: int, seed: int, node: int):
    """The quantizer applied to the raw slices of one node's gradient (bucket = slice of d entries), packed 4-bit:
    (q4 uint8 [S][d / 2], norms fp32 [S])."""
    g_node = _f32(g_node)
    d = int(layout.d)
    off, ln = _layers(layout)
    qs, ns, s0 = [], [], 0
    for o, m in zip(off, ln):
        S = int(m) // d
        if S == 0:
            continue
        q, nrm = quantize(g_node[int(o):int(o) + S * d].reshape(S, d), levels, seed, node, slice0=s0)
        qs.append(pack4(q)); ns.append(nrm)
        s0 += S
    if not qs:
        return np.zeros((0, d // 2), dtype=np.uint8), np.zeros(0, dtype=np.float32)
    return np.concatenate(qs), np.concatenate(ns)


def dequantize_raw4_aggregate(layout, q4_nodes, norms_nodes, g_nodes, levels: int, M: int) -> np.ndarray:
    """Sum over the nodes of the dequantised slices (double); tails: the plain sum of the raw tails.
    Entries outside every layer are NaN."""
    d = int(layout.d)
    off, ln = _layers(layout)
    out = np.full(M, np.nan, dtype=np.float64)
    s0 = 0
    for o, m in zip(off, ln):
        o, m = int(o), int(m)
        S = m // d
        acc = np.zeros((S, d), dtype=np.float64)
        for q4, nrm in zip(q4_nodes, norms_nodes):
            acc += unpack4(q4[s0:s0 + S]).astype(np.float64) * (nrm[s0:s0 + S].astype(np.float64)[:, None] / levels)
        out[o:o + S * d] = acc.ravel()
        out[o + S * d:o + m] = sum(_f32(g)[o + S * d:o + m].astype(np.float64) for g in g_nodes)
        s0 += S
    return out


def dequantize_aggregate(q_nodes, norms_nodes, levels: int):
    """Sum over the nodes of norm * q / levels, float64 [S][k]."""
    qs = [np.ascontiguousarray(q, dtype=np.int8) for q in q_nodes]
    ns = [_f32(n) for n in norms_nodes]
    S, k = qs[0].shape
    out = np.zeros((S, k), dtype=np.float64)
    qp = (ctypes.POINTER(ctypes.c_int8) * len(qs))(*[_p(q, ctypes.c_int8) for q in qs])
    npp = (ctypes.POINTER(ctypes.c_float) * len(ns))(*[_p(n, ctypes.c_float) for n in ns])
    rc = _load().gvqo_dequantize_aggregate(ctypes.c_int(k), ctypes.c_int64(S), ctypes.c_int(len(qs)), qp, npp,
                                           ctypes.c_int(levels), _p(out, ctypes.c_double))
    _check(rc, "dequantize_aggregate")
    return out


# --------------------------------------------------------------------------- whole path
def pipeline(layout, g_nodes, Ut, mu, M: int | None = None):
    """compress every node -> aggregate -> decompress (+ tails).  Returns (s_sum, g_hat) in float64."""
    N = len(g_nodes)
    M = int(g_nodes[0].size if M is None else M)
    s_nodes = [compress(layout, g, Ut, mu, N) for g in g_nodes]
    s_sum = aggregate(s_nodes)
    g_hat = decompress(layout, s_sum, Ut, mu, g_nodes, N, M)
    return s_sum, g_hat


def pipeline_quantized(layout, g_nodes, Ut, mu, levels: int, seed: int, M: int | None = None):
    """The path with the optional quantizer: compress every node (Eq. 3), round s_n to fp32 (what a node holds),
    quantize it with the node's index, sum the dequantised vectors (the compressed-domain aggregate of Eq. 4 over
    what the nodes transmit), decompress (Eq. 5, + tails).  Returns (s_sum, g_hat, q_nodes, norms_nodes)."""
    N = len(g_nodes)
    M = int(g_nodes[0].size if M is None else M)
    qs, ns = [], []
    for n, g in enumerate(g_nodes):
        q, nrm = quantize(compress(layout, g, Ut, mu, N).astype(np.float32), levels, seed, n)
        qs.append(q)
        ns.append(nrm)
    s_sum = dequantize_aggregate(qs, ns, levels)
    g_hat = decompress(layout, s_sum, Ut, mu, g_nodes, N, M)
    return s_sum, g_hat, qs, ns


# --------------------------------------------------------------------------- Algorithm 1
class SegmentLayout:
    """The part of a layout that one segment of Algorithm 1 covers: pieces of consecutive layers."""

    def __init__(self, d, k, piece_layer, layer_off, layer_len, slice0, slice1):
        self.d, self.k = int(d), int(k)
        self.piece_layer = list(piece_layer)         # layer of the parent layout that each piece was cut from
        self.first_layer = self.piece_layer[0] if self.piece_layer else 0
        self.layer_off, self.layer_len = list(layer_off), list(layer_len)
        self.slice0, self.slice1 = int(slice0), int(slice1)   # global slice range [slice0, slice1)

    @property
    def n_layers(self):
        return len(self.layer_len)


def segment_layout(layout, n_segments: int, j: int) -> SegmentLayout:
    """Algorithm 1, "partitions its g_n into N equal segments, each containing several gradient slices".

    Reading: segment j holds the global slices [floor(j S / G), floor((j + 1) S / G)), G = n_segments, S the
    number of full slices, counted through the layers in order; a layer cut by a boundary contributes a piece to
    both segments.  The uncompressed tail of a layer (and a layer shorter than one slice) travels with the
    segment that holds the slice just before it in that order (segment 0 if there is none).
    """
    d = int(layout.d)
    S = total_slices(layout)
    G = int(n_segments)
    lo, hi = (j * S) // G, ((j + 1) * S) // G

    def segment_of_slice(g):          # the segment whose range contains global slice g
        for jj in range(G):
            if (jj * S) // G <= g < ((jj + 1) * S) // G:
                return jj
        raise AssertionError(g)

    offs, lens, parents = [], [], []
    base = 0                           # global index of the layer's first slice
    for l, (o, m) in enumerate(zip(layout.layer_off, layout.layer_len)):
        o, m = int(o), int(m)
        Sl, tail = m // d, m % d
        a, b = max(lo, base), min(hi, base + Sl)          # this layer's slices that fall in the segment
        n_here = max(0, b - a)
        tail_here = False
        if tail > 0:
            before = base + Sl - 1                        # the slice just before the tail
            tail_here = (segment_of_slice(before) if before >= 0 else 0) == j
        if n_here > 0 or tail_here:
            start = o + (a - base) * d if n_here > 0 else o + Sl * d
            length = n_here * d + (tail if tail_here else 0)
            # a tail rides on the layer's last slices; if they belong to this segment the piece is contiguous
            assert not (tail_here and n_here > 0) or b == base + Sl
            offs.append(start)
            lens.append(length)
            parents.append(l)
        base += Sl
    return SegmentLayout(d, layout.k, parents, offs, lens, lo, hi)


def _segment_basis(layout, seg: SegmentLayout, Ut, mu):
    """Rows of (Ut, mu) for the pieces of a segment: a piece is compressed with the compressor of its layer."""
    return np.ascontiguousarray(Ut[seg.piece_layer]), np.ascontiguousarray(mu[seg.piece_layer])


def _segment_tails(seg: SegmentLayout, g: np.ndarray) -> np.ndarray:
    """The uncompressed entries of a segment's pieces (layer order), float64."""
    out = []
    for o, m in zip(seg.layer_off, seg.layer_len):
        full = (m // seg.d) * seg.d
        out.append(np.asarray(g[o + full:o + m], dtype=np.float64))
    return np.concatenate(out) if out else np.zeros(0)


def ring_allreduce(layout, g_nodes, Ut, mu, M: int | None = None):
    """Algorithm 1 simulated for N = len(g_nodes) nodes on a logical ring, one segment per node.

    A message is the pair (compressed slices of a segment [slices][k], its tail entries), float64.  Steps and
    indices are Algorithm 1's: node n first compresses segment n and sends it on; in step i = 1 .. N - 1 it
    receives segment [n - i] from node [n - 1], compresses its own segment [n - i], adds, and sends the sum to
    node [n + 1]; it then owns the complete segment [n + 1].  In step i = 0 .. N - 1 of the second round it
    decompresses segment [n + 1 - i] while receiving segment [n - i] (nothing is left to receive in the last
    step).  Returns (g_hat of every node: list of float64 [M], floats sent by every node: list of int).
    """
    N = len(g_nodes)
    M = int(g_nodes[0].size if M is None else M)
    segs = [segment_layout(layout, N, j) for j in range(N)]
    basis = [_segment_basis(layout, sg, Ut, mu) if sg.n_layers else (None, None) for sg in segs]

    def Q(n, j):                                    # Eq. 3 on node n's segment j, and its raw tails
        sg = segs[j]
        if sg.n_layers == 0:
            return np.zeros((0, int(layout.k))), np.zeros(0)
        return compress(sg, g_nodes[n], basis[j][0], basis[j][1], N), _segment_tails(sg, g_nodes[n])

    held = [dict() for _ in range(N)]              # held[n][j]: node n's current copy of compressed segment j
    sent = [0] * N
    inbox = [None] * N

    def send(n, j):
        s, t = held[n][j]
        inbox[(n + 1) % N] = (j, s.copy(), t.copy())
        sent[n] += s.size + t.size

    for n in range(N):
        held[n][n] = Q(n, n)
    if N > 1:                                      # a single node has no successor to send to
        for n in range(N):
            send(n, n)
    for i in range(1, N):
        arrived = list(inbox)
        for n in range(N):
            j = (n - i) % N
            jr, s_in, t_in = arrived[n]
            assert jr == j
            s_own, t_own = Q(n, j)
            held[n][j] = (s_in + s_own, t_in + t_own)
        if i < N - 1:
            for n in range(N):
                send(n, (n - i) % N)
    g_hat = [np.zeros(M, dtype=np.float64) for _ in range(N)]

    def decompress_into(n, j):
        sg = segs[j]
        if sg.n_layers == 0:
            return
        s, t = held[n][j]
        whole = SegmentLayout(sg.d, sg.k, sg.piece_layer, sg.layer_off, [(m // sg.d) * sg.d for m in sg.layer_len],
                              sg.slice0, sg.slice1)
        part = decompress(whole, s, basis[j][0], basis[j][1], None, N, M)  # Eq. 5 on the full slices only
        p = 0
        for o, m in zip(sg.layer_off, sg.layer_len):
            full = (m // sg.d) * sg.d
            g_hat[n][o:o + full] = part[o:o + full]
            g_hat[n][o + full:o + m] = t[p:p + m - full]
            p += m - full

    for i in range(N):
        if i < N - 1:
            for n in range(N):
                send(n, (n + 1 - i) % N)
        arrived = list(inbox)
        for n in range(N):
            decompress_into(n, (n + 1 - i) % N)
            if i < N - 1:
                jr, s_in, t_in = arrived[n]
                assert jr == (n - i) % N
                held[n][jr] = (s_in, t_in)
    return g_hat, sent
