"""CPU-side checks: the shared library loads and exports every declared symbol; host-only helpers."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_1811_03617_b200 import workloads as W

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def gvq():
    from paper_1811_03617_b200 import build, gvq as _gvq
    build.build()
    return _gvq


def test_library_exports_every_declared_symbol(gvq):
    header = (ROOT / "include" / "gvq.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(gvq_[a-z0-9_]+)\s*\(", header))
    assert {"gvq_fit_basis", "gvq_compress", "gvq_aggregate", "gvq_decompress", "gvq_quantize",
            "gvq_compress_aggregate"} <= declared
    lib = gvq.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in gvq.h but not exported"


def test_status_strings(gvq):
    lib = gvq.lib()
    seen = {lib.gvq_status_string(i).decode() for i in range(9)}
    assert len(seen) == 9 and "unknown status" not in seen
    assert lib.gvq_status_string(99).decode() == "unknown status"


def test_layout_check_and_counts(gvq):
    for f in W.WORKLOADS.values():
        w = f()
        h = gvq.HostLayout.of(w)
        assert h.check() == 0
        assert h.total_slices() == w.S and h.total_entries() == w.M
    H = gvq.HostLayout
    assert H(16, 4, [0], [64]).check() == 0
    assert H(16, 0, [0], [64]).check() == 2          # k < 1
    assert H(16, 17, [0], [64]).check() == 2         # k > d
    assert H(18, 4, [0], [64]).check() == 3          # d not a multiple of 4
    assert H(16, 4, [2], [64]).check() == 3          # offset not a multiple of 4
    assert H(16, 4, [0, 32], [64, 64]).check() == 2  # overlap
    assert H(16, 4, [64, 0], [64, 64]).check() == 2  # not sorted
    assert H(16, 4, [0], [-1]).check() == 2
    assert H(48, 4, [0], [480]).check() == 4         # no kernel for this d
    assert H(2048, 4, [0], [4096]).check() == 2      # d beyond the maximum
    assert H(1024, 128, [0], [4096]).check() == 4    # basis does not fit shared memory
    assert H(18, 4, [0], [64]).total_slices() == -1
    assert H(16, 4, [0], [64]).fit_workspace_bytes(0) == 0
    assert H(16, 4, [0], [64]).host_workspace_bytes(65) == 0
    a, b = H.of(W.resnet50()).fit_workspace_bytes(32), H.of(W.tiny()).fit_workspace_bytes(8)
    assert a > b > 0 and a % 256 == 0


def test_select_k_matches_oracle(gvq, oracle):
    rng = np.random.default_rng(0)
    for _ in range(50):
        d = int(rng.integers(1, 40))
        ev = np.sort(rng.exponential(1.0, d).astype(np.float32))[::-1].copy()
        lam = float(rng.uniform(0, 0.5))
        assert gvq.select_k(ev, lam) == oracle.select_k(ev.astype(np.float64), lam)
    out = ctypes.c_int32(-5)
    z = torch.zeros(6)
    assert gvq.lib().gvq_select_k(z.data_ptr(), 6, 0.01, ctypes.byref(out)) == 8 and out.value == 1
    assert gvq.lib().gvq_select_k(None, 6, 0.01, ctypes.byref(out)) == 1
    assert gvq.lib().gvq_select_k(z.data_ptr(), 6, 1.0, ctypes.byref(out)) == 2


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure path")
def test_no_gpu_fails_loudly(gvq):
    h = gvq.HostLayout.of(W.tiny())
    handle = ctypes.c_void_p()
    st = gvq.lib().gvq_create(ctypes.byref(handle), ctypes.byref(h.c), 0, None)
    assert st == 6 and not handle.value  # GVQ_ERR_CUDA, no context, no fallback
    with pytest.raises(RuntimeError):
        gvq.Context(W.tiny())


def test_workload_tables():
    expect = {"tiny": (1, 16384, 1024, 0), "resnet32": (32, 467632, 7306, 48), "vgg16": (13, 14710464, 114925, 64),
              "resnet50": (54, 25502912, 99620, 192), "large": (59, 99876864, 390144, 0)}
    for name, (nl, M, S, tail) in expect.items():
        w = W.WORKLOADS[name]()
        assert (w.n_layers, w.M, w.S, w.tail_entries) == (nl, M, S, tail)
        assert all(o % 4 == 0 for o in w.layer_off)
    w = W.resnet32()
    a, b = W.node_gradient(w, 3, iteration=2), W.node_gradient(w, 3, iteration=2)
    assert torch.equal(a, b) and not torch.equal(a, W.node_gradient(w, 4, iteration=2))
    # rank-k structure: the k + 1-th singular value of a layer's slices sits at the noise level
    X = a[w.layer_off[20]: w.layer_off[20] + w.layer_len[20]].view(-1, w.d)
    sv = torch.linalg.svdvals((X - X.mean(0)).double())
    assert sv[w.k - 1] > 5 * sv[w.k]


def test_schedule_follows_the_papers_plan(gvq):
    """Section 3: L_t uncompressed iterations, a fit, then at most L_c compressed ones; the compressed phase ends
    early when the majority of the nodes is over the loss threshold (Eq. 7)."""
    import torch
    L_t, L_c, N, layers = 3, 5, 4, 2
    sch = gvq.Schedule(L_t, L_c, N, 0.1)
    assert sch.phase == gvq.PHASE_COLLECT
    assert [sch.step() for _ in range(L_t)] == [gvq.ACT_NONE, gvq.ACT_NONE, gvq.ACT_FIT]
    assert sch.phase == gvq.PHASE_COMPRESS

    def monitor(rel_loss_per_node):
        m = torch.zeros((layers, 2, N), dtype=torch.float64)
        m[:, 0, :] = 10.0                                   # energy per layer
        for n, r in enumerate(rel_loss_per_node):
            m[:, 1, n] = 10.0 * (1.0 - r)                   # captured
        return m

    # all nodes fine: runs the full L_c, with and without a monitor
    acts = [sch.step(monitor([0.01] * N) if i % 2 == 0 else None) for i in range(L_c)]
    assert acts == [gvq.ACT_NONE] * (L_c - 1) + [gvq.ACT_RESTART]
    assert sch.phase == gvq.PHASE_COLLECT and sch.counters() == {"iteration": L_t + L_c, "refreshes": 1, "early_stops": 0}
    assert [sch.step() for _ in range(L_t)][-1] == gvq.ACT_FIT
    # exactly half of the nodes over: not a majority
    assert sch.step(monitor([0.5, 0.5, 0.01, 0.01])) == gvq.ACT_NONE and sch.nodes_over == 2
    # three of four over: stop early
    assert sch.step(monitor([0.5, 0.5, 0.11, 0.01])) == gvq.ACT_RESTART and sch.nodes_over == 3
    assert sch.phase == gvq.PHASE_COLLECT and sch.counters()["early_stops"] == 1
    # the threshold is strict and relative to the energy summed over the layers
    for _ in range(L_t):
        sch.step()
    assert sch.step(monitor([0.1, 0.1, 0.1, 0.1])) == gvq.ACT_NONE and sch.nodes_over == 0
    with pytest.raises(gvq.GvqError):
        gvq.Schedule(0, 5, 4, 0.1)
    with pytest.raises(gvq.GvqError):
        gvq.Schedule(3, 5, 4, 1.5)
    sch.close()


@pytest.mark.parametrize("kind,n_nodes", [(0, 16), (0, 1), (0, 64), (1, 16)])
def test_work_partition_is_a_balanced_cover(gvq, kind, n_nodes):
    """The split of the tensor-core kernels' work units over the CTAs: contiguous, complete, no empty part before
    a non-empty one, and no part much above the mean cost under the documented model."""
    for w, parts in ((W.resnet50(), 148), (W.vgg16(), 148), (W.resnet32(), 148),
                     (W.custom("few", 5, d=128, k=16, N=4, L=1, layer_len=[128 * 130, 128 * 3, 128 * 700]), 7)):
        start, total = gvq.work_partition(w, kind, n_nodes, parts)
        per_tile = n_nodes if kind == 0 else (w.d + 127) // 128
        tiles_layer = [l for l, m in enumerate(w.layer_len) for _ in range(0, m // w.d, 128)]
        assert total == len(tiles_layer) * per_tile
        assert len(start) == parts + 1 and start[0] == 0 and start[-1] == total
        sizes = [b - a for a, b in zip(start, start[1:])]
        assert all(s >= 0 for s in sizes)
        nonempty = [i for i, s in enumerate(sizes) if s > 0]
        assert nonempty == list(range(len(nonempty))), "empty parts only at the end"
        stage = 2.0 if kind == 0 else 4.0

        def cost(a, b):
            layers = {tiles_layer[u // per_tile] for u in range(a, b)}
            return (b - a) + stage * len(layers)
        costs = [cost(a, b) for a, b in zip(start, start[1:]) if b > a]
        n_layers_present = len(set(tiles_layer))
        lower = (total + stage * n_layers_present) / parts          # no split can beat the mean
        assert max(costs) <= lower + stage + 1.0 + 1e-6 or total <= parts


def test_packed_floats_counts_the_kept_coordinates():
    """gvq_packed_floats (host only): sum_l S_l * k_l + the tail entries; bad lengths are refused."""
    import ctypes
    from paper_1811_03617_b200 import gvq, workloads as W
    w = W.custom("packed", 5, d=16, k=4, N=2, L=1, layer_len=[16 * 10 + 3, 7, 16 * 5], layer_off=[0, 164, 172])
    hl = gvq.HostLayout.of(w)
    assert hl.packed_floats([4, 4, 4]) == hl.exchange_floats() == 15 * 4 + 10
    assert hl.packed_floats([1, 3, 0]) == 10 * 1 + 0 + 0 + 10
    assert hl.packed_floats([5, 0, 0]) == -1 and hl.packed_floats([-1, 0, 0]) == -1
    assert gvq.lib().gvq_packed_floats(ctypes.byref(hl.c), None) == -1
