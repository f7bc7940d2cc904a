"""Comparison helpers shared by the tests (no method arithmetic: norms and angles only)."""
import numpy as np


def rel_l2(got, want) -> float:
    got = np.asarray(got, dtype=np.float64).ravel()
    want = np.asarray(want, dtype=np.float64).ravel()
    den = np.linalg.norm(want)
    num = np.linalg.norm(got - want)
    return float(num / den) if den > 0 else float(num)


def subspace_angle(Ut_a, Ut_b) -> float:
    """Largest principal angle between the row spaces of two [k][d] matrices (rows ~orthonormal)."""
    A = np.asarray(Ut_a, dtype=np.float64)
    B = np.asarray(Ut_b, dtype=np.float64)
    Qb, _ = np.linalg.qr(B.T)
    Qa, _ = np.linalg.qr(A.T)
    R = Qa - Qb @ (Qb.T @ Qa)          # component of span(A) outside span(B)
    s = np.linalg.svd(R, compute_uv=False)
    return float(np.arcsin(min(1.0, s.max())))


def layer_slices(w, l):
    """(flat-gradient range of the full slices, compressed-buffer row range, tail range) of layer l."""
    off, m = w.layer_off[l], w.layer_len[l]
    S = m // w.d
    soff = sum(x // w.d for x in w.layer_len[:l])
    return (off, off + S * w.d), (soff, soff + S), (off + S * w.d, off + m)
