"""Seeded synthetic workloads shaped like the CNN gradients GradiVeQ compresses.

This module only *describes* workloads (layer tables, sizes) and *draws* their
inputs.  It holds none of the method's arithmetic and imports neither the CUDA
binding nor any checker, so tests and benchmarks can hand the very same bytes
to every implementation they compare.

Input recipe (stand-in for recorded ResNet/VGG gradients, which show strong
linear correlation inside a slice -- the paper's "linear correlation" and
"spatial domain consistency" observations): for layer l with slice length d and
rank k,

    node slice  x = mu_l + A_l z + eps,   z ~ N(0, I_k),  eps ~ N(0, sigma_l^2 I_d)

with mu_l ~ N(0, 0.3^2)^d, A_l ~ N(0, 1)^{d x k} fixed per (workload, layer),
sigma_l = 0.01 (absolute, "tiny") or 0.05 * sqrt(||A_l||_F^2 / d) (relative).
Entries of a layer past its last full slice ("tail") are N(0, 1).
A stored, aggregated gradient (the samples of a basis fit) is either the literal
sum of N node draws or, for the large workloads, one draw of
N mu + sqrt(N) (A z + eps), which has the same distribution.
With drift, A_l(t) = cos(theta t) A_l + sin(theta t) B_l, B_l an independent
Gaussian matrix, theta = 1e-3 rad per iteration.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Sequence

import torch

BASE_SEED = 20181103

# purposes of a random stream
_P_MU, _P_A, _P_B, _P_NODE, _P_STORED, _P_TAIL = 1, 2, 3, 4, 5, 6


@dataclass
class Workload:
    """A gradient layout plus the parameters of its synthetic inputs."""
    name: str
    ident: int                      # enters every seed
    d: int                          # slice length
    k: int                          # compressed length / rank of the synthetic signal
    N: int                          # simulated nodes
    L: int                          # stored gradients used by a basis fit
    layer_len: List[int]
    sigma_abs: float | None = None  # absolute noise std; None -> 0.05 relative
    drift: float = 0.0              # rad per iteration
    literal_sums: bool = False      # stored gradients are literal sums of N node draws
    layer_off: List[int] = field(default_factory=list)

    def __post_init__(self):
        if not self.layer_off:
            off, acc = [], 0
            for m in self.layer_len:
                off.append(acc)
                acc += m
            self.layer_off = off

    @property
    def n_layers(self) -> int:
        return len(self.layer_len)

    @property
    def M(self) -> int:
        return max((o + m for o, m in zip(self.layer_off, self.layer_len)), default=0)

    @property
    def slices_per_layer(self) -> List[int]:
        return [m // self.d for m in self.layer_len]

    @property
    def S(self) -> int:
        return sum(self.slices_per_layer)

    @property
    def tail_entries(self) -> int:
        return sum(m % self.d for m in self.layer_len)

    def stream_bytes(self) -> int:
        """Algorithmic bytes of one compress + N-sum + decompress pass: every node's
        gradient read once, the aggregate written once."""
        return (self.N + 1) * self.M * 4


def _resnet32_layers() -> List[int]:
    ls = [3 * 3 * 3 * 16]
    ls += [3 * 3 * 16 * 16] * 10
    ls += [3 * 3 * 16 * 32] + [3 * 3 * 32 * 32] * 9
    ls += [3 * 3 * 32 * 64] + [3 * 3 * 64 * 64] * 9
    ls += [64 * 100]
    return ls


def _vgg16_layers() -> List[int]:
    ch = [3, 64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512]
    return [9 * ch[i] * ch[i + 1] for i in range(13)]


def _resnet50_layers() -> List[int]:
    ls = [7 * 7 * 3 * 64]
    cin = 64
    for w, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            ls += [cin * w, 9 * w * w, w * 4 * w]
            if b == 0:
                ls.append(cin * 4 * w)
            cin = 4 * w
    ls.append(2048 * 1000)
    return ls


def _large_layers() -> List[int]:
    ls: List[int] = []
    for _ in range(29):
        ls += [1024 * 1024, 9 * 512 * 512]
    ls.append(1024 * 1024)
    return ls


def tiny() -> Workload:
    return Workload("tiny", 1, d=16, k=4, N=4, L=8, layer_len=[16384], sigma_abs=0.01, literal_sums=True)


def resnet32() -> Workload:
    return Workload("resnet32", 2, d=64, k=8, N=8, L=8, layer_len=_resnet32_layers(), literal_sums=True)


def vgg16() -> Workload:
    return Workload("vgg16", 3, d=128, k=16, N=16, L=8, layer_len=_vgg16_layers())


def resnet50() -> Workload:
    return Workload("resnet50", 4, d=256, k=32, N=16, L=32, layer_len=_resnet50_layers(), drift=1e-3)


def large() -> Workload:
    return Workload("large", 5, d=256, k=32, N=32, L=8, layer_len=_large_layers())


WORKLOADS = {"tiny": tiny, "resnet32": resnet32, "vgg16": vgg16, "resnet50": resnet50, "large": large}


def custom(name: str, ident: int, d: int, k: int, N: int, L: int, layer_len: Sequence[int], **kw) -> Workload:
    """A hand-made layout for edge-case tests (ragged tails, layers shorter than a slice, ...)."""
    return Workload(name, ident, d=d, k=k, N=N, L=L, layer_len=list(layer_len), **kw)


# --------------------------------------------------------------------------- random streams
def _gen(device, *key: int) -> torch.Generator:
    """A generator whose seed is a fixed integer mix of (BASE_SEED, *key)."""
    h = BASE_SEED
    for v in key:
        h = (h * 6364136223846793005 + (int(v) + 1) * 1442695040888963407) % (1 << 63)
        h ^= h >> 29
    g = torch.Generator(device=device)
    g.manual_seed(h % (1 << 62))
    return g


def _randn(shape, device, *key) -> torch.Tensor:
    return torch.randn(shape, generator=_gen(device, *key), device=device, dtype=torch.float32)


def layer_params(w: Workload, layer: int, device="cpu", iteration: int = 0):
    """(mu_l [d], A_l(t) [d][k], sigma_l) of one layer; always drawn on the CPU so that they
    do not depend on the device the data are generated on."""
    mu = 0.3 * _randn((w.d,), "cpu", w.ident, layer, _P_MU)
    A = _randn((w.d, w.k), "cpu", w.ident, layer, _P_A)
    rho2 = float((A.double() ** 2).sum() / w.d)
    if w.drift != 0.0 and iteration != 0:
        B = _randn((w.d, w.k), "cpu", w.ident, layer, _P_B)
        th = w.drift * iteration
        A = math.cos(th) * A + math.sin(th) * B
    sigma = w.sigma_abs if w.sigma_abs is not None else 0.05 * math.sqrt(rho2)
    return mu.to(device), A.to(device), sigma


def _draw_layer(w: Workload, layer: int, out: torch.Tensor, scale_mu: float, scale_rest: float,
                iteration: int, *key: int) -> None:
    """Fill out[layer_off : layer_off + layer_len] with scale_mu * mu + scale_rest * (A z + eps)."""
    dev = out.device
    off, m = w.layer_off[layer], w.layer_len[layer]
    S, tail = m // w.d, m % w.d
    if S > 0:
        mu, A, sigma = layer_params(w, layer, dev, iteration)
        g = _gen(dev, w.ident, layer, *key)
        z = torch.randn((S, w.k), generator=g, device=dev, dtype=torch.float32)
        x = out[off: off + S * w.d].view(S, w.d)
        x.normal_(0.0, sigma, generator=g)
        x.addmm_(z, A.t())
        if scale_rest != 1.0:
            x.mul_(scale_rest)
        x.add_(scale_mu * mu)
    if tail > 0:
        out[off + S * w.d: off + m] = _randn((tail,), dev, w.ident, layer, _P_TAIL, *key)


def node_gradient(w: Workload, node: int, iteration: int = 0, device="cpu", out: torch.Tensor | None = None):
    """One node's flat fp32 gradient [M] at a training iteration."""
    if out is None:
        out = torch.zeros(w.M, dtype=torch.float32, device=device)
    for l in range(w.n_layers):
        _draw_layer(w, l, out, 1.0, 1.0, iteration, _P_NODE, node, iteration)
    return out


def node_gradients(w: Workload, iteration: int = 0, device="cpu") -> List[torch.Tensor]:
    return [node_gradient(w, n, iteration, device) for n in range(w.N)]


def stored_gradients(w: Workload, L: int | None = None, device="cpu", first_iteration: int = 0) -> torch.Tensor:
    """[L][M] aggregated gradients of iterations first_iteration .. first_iteration + L - 1."""
    L = w.L if L is None else L
    hist = torch.zeros((L, w.M), dtype=torch.float32, device=device)
    for h in range(L):
        it = first_iteration + h
        if w.literal_sums:
            tmp = torch.zeros(w.M, dtype=torch.float32, device=device)
            for n in range(w.N):
                tmp.zero_()
                for l in range(w.n_layers):
                    _draw_layer(w, l, tmp, 1.0, 1.0, it, _P_STORED, n, it)
                hist[h] += tmp
        else:
            for l in range(w.n_layers):
                _draw_layer(w, l, hist[h], float(w.N), math.sqrt(w.N), it, _P_STORED, it)
    return hist


def random_basis(w: Workload, device="cpu", seed_key: int = 0):
    """An orthonormal Ut [layers][k][d] and a mu [layers][d] that are NOT fitted: QR of a
    Gaussian matrix mixed with the layer's A so that the projections are not tiny."""
    Ut = torch.empty((w.n_layers, w.k, w.d), dtype=torch.float32)
    mu = torch.empty((w.n_layers, w.d), dtype=torch.float32)
    for l in range(w.n_layers):
        m, A, _ = layer_params(w, l, "cpu")
        G = A.double() + 0.1 * _randn((w.d, w.k), "cpu", w.ident, l, 77, seed_key).double()
        Q, _ = torch.linalg.qr(G)
        Ut[l] = Q.t().float()
        mu[l] = w.N * m + 0.01 * _randn((w.d,), "cpu", w.ident, l, 78, seed_key)
    return Ut.to(device), mu.to(device)
