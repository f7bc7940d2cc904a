"""Thin ctypes binding of libgvq.so: argument marshalling only.

Every function here has the name and the meaning of the C entry point it calls
(see include/gvq.h); tensors are torch CUDA tensors used purely as device
memory, and the current torch stream is handed to the library.  There is no
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Sequence

import torch

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libgvq.so"
_lib = None

MAX_NODES = 64

STATUS = {0: "GVQ_OK", 1: "GVQ_ERR_NULL", 2: "GVQ_ERR_SHAPE", 3: "GVQ_ERR_ALIGN", 4: "GVQ_ERR_UNSUPPORTED",
          5: "GVQ_ERR_WORKSPACE", 6: "GVQ_ERR_CUDA", 7: "GVQ_ERR_NOT_CONVERGED", 8: "GVQ_ERR_DEGENERATE",
          9: "GVQ_ERR_TIMEOUT", 10: "GVQ_ERR_CAPTURE"}


class GvqError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().gvq_status_string(status).decode()
        super().__init__(f"{what}: {STATUS.get(status, status)} ({msg})")


class _Layout(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("k", ctypes.c_int32), ("n_layers", ctypes.c_int32),
                ("layer_off", ctypes.POINTER(ctypes.c_int64)), ("layer_len", ctypes.POINTER(ctypes.c_int64))]


def lib() -> ctypes.CDLL:
    """Loads libgvq.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_1811_03617_b200.build` "
                               "(there is no fallback implementation)")
        L = ctypes.CDLL(str(LIB_PATH))
        vp, i32, i64, u64, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32
        LP = ctypes.POINTER(_Layout)
        L.gvq_status_string.restype = ctypes.c_char_p
        L.gvq_status_string.argtypes = [i32]
        L.gvq_layout_check.argtypes = [LP]
        L.gvq_total_slices.restype = i64
        L.gvq_total_slices.argtypes = [LP]
        L.gvq_total_entries.restype = i64
        L.gvq_total_entries.argtypes = [LP]
        L.gvq_fit_workspace_bytes.restype = ctypes.c_size_t
        L.gvq_fit_workspace_bytes.argtypes = [LP, i32]
        L.gvq_host_workspace_bytes.restype = ctypes.c_size_t
        L.gvq_host_workspace_bytes.argtypes = [LP, i32]
        L.gvq_select_k.argtypes = [vp, i32, ctypes.c_double, ctypes.POINTER(ctypes.c_int32)]
        L.gvq_create.argtypes = [ctypes.POINTER(vp), LP, i32, vp]
        L.gvq_destroy.argtypes = [vp]
        L.gvq_set_stream.argtypes = [vp, vp]
        L.gvq_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
        L.gvq_last_cuda_error.argtypes = [vp]
        L.gvq_set_projection_path.argtypes = [vp, i32]
        L.gvq_set_fit_path.argtypes = [vp, i32]
        L.gvq_device_status.argtypes = [vp]
        L.gvq_compress.argtypes = [vp, vp, vp, vp, i32, vp]
        L.gvq_aggregate.argtypes = [vp, vp, i32, vp]
        L.gvq_compress_aggregate.argtypes = [vp, vp, i32, vp, vp, vp, vp]
        L.gvq_compress_quantize_aggregate.argtypes = [vp, vp, i32, vp, vp, i32, u64, vp, vp, vp]
        L.gvq_decompress.argtypes = [vp, vp, vp, vp, vp, i32, vp]
        L.gvq_fit_basis.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
        L.gvq_refresh_basis.argtypes = [vp, vp, i64, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        L.gvq_fit_basis_static.argtypes = [vp, vp, i64, i32, i32, i32, vp, vp, vp, vp]
        L.gvq_fit_moments_count.restype = i64
        L.gvq_fit_moments_count.argtypes = [LP]
        L.gvq_fit_centre.argtypes = [vp, vp, i64, i32, vp]
        L.gvq_fit_moments.argtypes = [vp, vp, i64, i32, vp, vp]
        L.gvq_fit_from_moments.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp]
        L.gvq_quantize.argtypes = [vp, vp, i32, u64, u32, vp, vp]
        L.gvq_compress_aggregate_monitored.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
        L.gvq_quantize_aggregate.argtypes = [vp, vp, i32, i32, u64, vp, vp, vp]
        L.gvq_dequantize_aggregate.argtypes = [vp, vp, vp, i32, i32, vp]
        L.gvq_allreduce_host.argtypes = [vp, vp, i32, vp, vp, vp]
        L.gvq_allreduce_host_quantized.argtypes = [vp, vp, i32, vp, vp, i32, u64, vp]
        L.gvq_host_prepare.argtypes = [vp]
        L.gvq_set_limits.argtypes = [vp, i32, i64]
        L.gvq_test_drop_load.argtypes = [vp, i32]
        L.gvq_work_partition.argtypes = [LP, i32, i32, i32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(i64)]
        L.gvq_quantize_raw4.argtypes = [vp, vp, i32, u64, u32, vp, vp]
        L.gvq_quantize_raw4_aggregate.argtypes = [vp, vp, i32, i32, u64, vp, vp, vp]
        L.gvq_dequantize_raw4_aggregate.argtypes = [vp, vp, vp, vp, i32, i32, vp]
        L.gvq_flatten_layer.argtypes = [vp, vp, vp, i32, i32, i32]
        L.gvq_unflatten_layer.argtypes = [vp, vp, vp, i32, i32, i32]
        L.gvq_exchange_floats.argtypes = [LP]
        L.gvq_exchange_floats.restype = i64
        L.gvq_segment_layout.argtypes = [LP, i32, i32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32),
                                         ctypes.POINTER(i64), ctypes.POINTER(i64)]
        L.gvq_compress_aggregate_partial.argtypes = [vp, vp, i32, i32, vp, vp, vp]
        L.gvq_exchange_accumulate.argtypes = [vp, vp, vp]
        L.gvq_decompress_exchanged.argtypes = [vp, vp, vp, vp, vp]
        L.gvq_mask_basis.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.gvq_packed_floats.restype = i64
        L.gvq_packed_floats.argtypes = [LP, ctypes.POINTER(ctypes.c_int32)]
        L.gvq_set_layer_k.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
        L.gvq_exchange_pack.argtypes = [vp, vp, vp]
        L.gvq_exchange_unpack.argtypes = [vp, vp, vp]
        L.gvq_schedule_create.argtypes = [ctypes.POINTER(vp), i32, i32, i32, ctypes.c_double]
        L.gvq_schedule_destroy.argtypes = [vp]
        L.gvq_schedule_phase.argtypes = [vp]
        L.gvq_schedule_nodes_over.argtypes = [vp]
        L.gvq_schedule_step.argtypes = [vp, vp, i32, ctypes.POINTER(i32)]
        L.gvq_schedule_counters.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i64)]
        _lib = L
    return _lib


def _ptr_array(tensors: Sequence[torch.Tensor]):
    return (ctypes.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def _check(status: int, what: str) -> None:
    if status != 0:
        raise GvqError(status, what)


class HostLayout:
    """Owns the ctypes image of a gvq_layout (host-only helpers work without a GPU)."""

    def __init__(self, d: int, k: int, layer_off: Sequence[int], layer_len: Sequence[int]):
        n = len(layer_len)
        self.d, self.k = int(d), int(k)
        self.layer_off, self.layer_len = [int(v) for v in layer_off], [int(v) for v in layer_len]
        self._off = (ctypes.c_int64 * n)(*self.layer_off)
        self._len = (ctypes.c_int64 * n)(*self.layer_len)
        self.c = _Layout(self.d, self.k, n, self._off, self._len)

    @classmethod
    def of(cls, w) -> "HostLayout":
        return cls(w.d, w.k, w.layer_off, w.layer_len)

    def check(self) -> int:
        return lib().gvq_layout_check(ctypes.byref(self.c))

    def total_slices(self) -> int:
        return lib().gvq_total_slices(ctypes.byref(self.c))

    def total_entries(self) -> int:
        return lib().gvq_total_entries(ctypes.byref(self.c))

    def fit_workspace_bytes(self, L: int) -> int:
        return lib().gvq_fit_workspace_bytes(ctypes.byref(self.c), L)

    def host_workspace_bytes(self, N: int) -> int:
        return lib().gvq_host_workspace_bytes(ctypes.byref(self.c), N)

    def exchange_floats(self) -> int:
        return lib().gvq_exchange_floats(ctypes.byref(self.c))

    def fit_moments_count(self) -> int:
        return lib().gvq_fit_moments_count(ctypes.byref(self.c))

    def packed_floats(self, k_per_layer) -> int:
        ks = (ctypes.c_int32 * len(self.layer_len))(*[int(x) for x in k_per_layer])
        return lib().gvq_packed_floats(ctypes.byref(self.c), ks)


def segment_layout(layout, n_segments: int, j: int):
    """gvq_segment_layout: (HostLayout of segment j or None when it is empty, parent layer of each piece)."""
    hl = layout if isinstance(layout, HostLayout) else HostLayout.of(layout)
    n = len(hl.layer_len)
    n_pieces = ctypes.c_int32(0)
    layer = (ctypes.c_int32 * n)()
    off, ln = (ctypes.c_int64 * n)(), (ctypes.c_int64 * n)()
    _check(lib().gvq_segment_layout(ctypes.byref(hl.c), n_segments, j, ctypes.byref(n_pieces), layer, off, ln),
           "gvq_segment_layout")
    m = n_pieces.value
    if m == 0:
        return None, []
    return HostLayout(hl.d, hl.k, list(off[:m]), list(ln[:m])), list(layer[:m])


def work_partition(layout, kind: int, n_nodes: int, n_parts: int):
    """gvq_work_partition: (list of n_parts + 1 unit indices, total units)."""
    hl = layout if isinstance(layout, HostLayout) else HostLayout.of(layout)
    start = (ctypes.c_int32 * (n_parts + 1))()
    total = ctypes.c_int64(0)
    _check(lib().gvq_work_partition(ctypes.byref(hl.c), kind, n_nodes, n_parts, start, ctypes.byref(total)),
           "gvq_work_partition")
    return list(start), total.value


def select_k(evals, lambda_loss: float) -> int:
    """gvq_select_k (Eq. 6) on one layer's descending eigenvalues (host tensor / sequence)."""
    ev = torch.as_tensor(evals, dtype=torch.float32).contiguous().cpu()
    out = ctypes.c_int32(0)
    _check(lib().gvq_select_k(ev.data_ptr(), ev.numel(), float(lambda_loss), ctypes.byref(out)), "gvq_select_k")
    return out.value


PHASE_COLLECT, PHASE_COMPRESS = 0, 1
ACT_NONE, ACT_FIT, ACT_RESTART = 0, 1, 2


class Schedule:
    """gvq_schedule: the collect / fit / compress plan with the majority rule on Eq. 7's loss (host only)."""

    def __init__(self, L_t: int, L_c: int, n_nodes: int, loss_threshold: float):
        self._h = ctypes.c_void_p()
        _check(lib().gvq_schedule_create(ctypes.byref(self._h), L_t, L_c, n_nodes, float(loss_threshold)),
               "gvq_schedule_create")

    def close(self):
        if self._h:
            lib().gvq_schedule_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def phase(self) -> int:
        return lib().gvq_schedule_phase(self._h)

    @property
    def nodes_over(self) -> int:
        return lib().gvq_schedule_nodes_over(self._h)

    def step(self, monitor_host: Optional[torch.Tensor] = None) -> int:
        """Call after every iteration; monitor_host: None or a CPU float64 tensor [n_layers][2][n_nodes]."""
        action = ctypes.c_int(0)
        ptr, n_layers = None, 0
        if monitor_host is not None:
            assert monitor_host.dtype == torch.float64 and not monitor_host.is_cuda and monitor_host.is_contiguous()
            ptr, n_layers = monitor_host.data_ptr(), monitor_host.shape[0]
        _check(lib().gvq_schedule_step(self._h, ptr, n_layers, ctypes.byref(action)), "gvq_schedule_step")
        return action.value

    def counters(self):
        a, b, c = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
        _check(lib().gvq_schedule_counters(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
               "gvq_schedule_counters")
        return {"iteration": a.value, "refreshes": b.value, "early_stops": c.value}


class Context:
    """gvq_ctx for one layout on one CUDA device."""

    def __init__(self, layout, device: Optional[int] = None):
        self.layout = layout if isinstance(layout, HostLayout) else HostLayout.of(layout)
        if not torch.cuda.is_available():
            raise RuntimeError("gvq needs a CUDA device (there is no CPU fallback)")
        self.device = torch.cuda.current_device() if device is None else int(device)
        self._h = ctypes.c_void_p()
        st = lib().gvq_create(ctypes.byref(self._h), ctypes.byref(self.layout.c), self.device, self._stream())
        _check(st, "gvq_create")
        self.d, self.k = self.layout.d, self.layout.k
        self.S = self.layout.total_slices()
        self.M = self.layout.total_entries()
        self.n_layers = len(self.layout.layer_len)
        self._ws = None

    def _stream(self):
        return ctypes.c_void_p(torch.cuda.current_stream(self.device).cuda_stream)

    def _sync_stream(self):
        _check(lib().gvq_set_stream(self._h, self._stream()), "gvq_set_stream")

    def close(self):
        if self._h:
            lib().gvq_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_projection_path(self, path: int):
        _check(lib().gvq_set_projection_path(self._h, path), "gvq_set_projection_path")

    def set_fit_path(self, path: int):
        _check(lib().gvq_set_fit_path(self._h, path), "gvq_set_fit_path")

    def set_limits(self, max_sweeps: int = 0, wait_cycles: int = 0):
        """gvq_set_limits (testing hook): 0 restores a default."""
        _check(lib().gvq_set_limits(self._h, int(max_sweeps), int(wait_cycles)), "gvq_set_limits")

    def test_drop_load(self, on: bool):
        _check(lib().gvq_test_drop_load(self._h, 1 if on else 0), "gvq_test_drop_load")

    def device_status(self):
        self._sync_stream()
        _check(lib().gvq_device_status(self._h), "gvq_device_status")

    def set_workspace(self, ws: Optional[torch.Tensor]):
        self._ws = ws
        if ws is None:
            _check(lib().gvq_set_workspace(self._h, None, 0), "gvq_set_workspace")
        else:
            _check(lib().gvq_set_workspace(self._h, ws.data_ptr(), ws.numel() * ws.element_size()),
                   "gvq_set_workspace")

    def ensure_workspace(self, nbytes: int):
        if self._ws is None or self._ws.numel() < nbytes:
            self.set_workspace(torch.empty(max(nbytes, 256), dtype=torch.uint8, device=f"cuda:{self.device}"))

    # ---- hot path -------------------------------------------------------------------------
    def compress(self, g_node, Ut, mu, N, s_node):
        self._sync_stream()
        _check(lib().gvq_compress(self._h, g_node.data_ptr(), Ut.data_ptr(), mu.data_ptr(), N, s_node.data_ptr()),
               "gvq_compress")

    def aggregate(self, s_nodes, s_sum):
        self._sync_stream()
        _check(lib().gvq_aggregate(self._h, _ptr_array(s_nodes), len(s_nodes), s_sum.data_ptr()), "gvq_aggregate")

    def compress_aggregate(self, g_nodes, Ut, mu, s_sum, s_nodes=None):
        self._sync_stream()
        sn = _ptr_array(s_nodes) if s_nodes is not None else None
        _check(lib().gvq_compress_aggregate(self._h, _ptr_array(g_nodes), len(g_nodes), Ut.data_ptr(),
                                            mu.data_ptr(), s_sum.data_ptr(), sn), "gvq_compress_aggregate")

    def compress_aggregate_partial(self, g_nodes, N, Ut, mu, x):
        self._sync_stream()
        _check(lib().gvq_compress_aggregate_partial(self._h, _ptr_array(g_nodes), len(g_nodes), N, Ut.data_ptr(),
                                                    mu.data_ptr(), x.data_ptr()), "gvq_compress_aggregate_partial")

    def exchange_accumulate(self, x_acc, x_in):
        self._sync_stream()
        _check(lib().gvq_exchange_accumulate(self._h, x_acc.data_ptr(), x_in.data_ptr()), "gvq_exchange_accumulate")

    def decompress_exchanged(self, x, Ut, mu, g_hat):
        self._sync_stream()
        _check(lib().gvq_decompress_exchanged(self._h, x.data_ptr(), Ut.data_ptr(), mu.data_ptr(), g_hat.data_ptr()),
               "gvq_decompress_exchanged")

    def quantize_raw4(self, g_node, levels, seed, node, q4, norms):
        self._sync_stream()
        _check(lib().gvq_quantize_raw4(self._h, g_node.data_ptr(), levels, seed, node, q4.data_ptr(), norms.data_ptr()),
               "gvq_quantize_raw4")

    def quantize_raw4_aggregate(self, g_nodes, levels, seed, g_sum, q4_nodes=None, norms_nodes=None):
        self._sync_stream()
        qp = _ptr_array(q4_nodes) if q4_nodes is not None else None
        npp = _ptr_array(norms_nodes) if norms_nodes is not None else None
        _check(lib().gvq_quantize_raw4_aggregate(self._h, _ptr_array(g_nodes), len(g_nodes), levels, seed,
                                                 g_sum.data_ptr(), qp, npp), "gvq_quantize_raw4_aggregate")

    def dequantize_raw4_aggregate(self, q4_nodes, norms_nodes, g_nodes_for_tails, levels, g_sum):
        self._sync_stream()
        gp = _ptr_array(g_nodes_for_tails) if g_nodes_for_tails is not None else None
        _check(lib().gvq_dequantize_raw4_aggregate(self._h, _ptr_array(q4_nodes), _ptr_array(norms_nodes), gp, levels,
                                                   len(q4_nodes), g_sum.data_ptr()), "gvq_dequantize_raw4_aggregate")

    def flatten_layer(self, framework, flat, F, D, X):
        self._sync_stream()
        _check(lib().gvq_flatten_layer(self._h, framework.data_ptr(), flat.data_ptr(), F, D, X), "gvq_flatten_layer")

    def unflatten_layer(self, flat, framework, F, D, X):
        self._sync_stream()
        _check(lib().gvq_unflatten_layer(self._h, flat.data_ptr(), framework.data_ptr(), F, D, X), "gvq_unflatten_layer")

    def mask_basis(self, Ut, k_per_layer):
        ks = (ctypes.c_int32 * self.n_layers)(*[int(x) for x in k_per_layer])
        self._sync_stream()
        _check(lib().gvq_mask_basis(self._h, Ut.data_ptr(), ks), "gvq_mask_basis")

    def set_layer_k(self, k_per_layer):
        """gvq_set_layer_k: per-layer compressed lengths for exchange_pack / exchange_unpack (None = all k)."""
        self._sync_stream()
        ks = None if k_per_layer is None else (ctypes.c_int32 * self.n_layers)(*[int(x) for x in k_per_layer])
        _check(lib().gvq_set_layer_k(self._h, ks), "gvq_set_layer_k")

    def exchange_pack(self, x, x_packed):
        self._sync_stream()
        _check(lib().gvq_exchange_pack(self._h, x.data_ptr(), x_packed.data_ptr()), "gvq_exchange_pack")

    def exchange_unpack(self, x_packed, x):
        self._sync_stream()
        _check(lib().gvq_exchange_unpack(self._h, x_packed.data_ptr(), x.data_ptr()), "gvq_exchange_unpack")

    def compress_aggregate_monitored(self, g_nodes, Ut, mu, s_sum, monitor, s_nodes=None):
        self._sync_stream()
        sn = _ptr_array(s_nodes) if s_nodes is not None else None
        _check(lib().gvq_compress_aggregate_monitored(self._h, _ptr_array(g_nodes), len(g_nodes), Ut.data_ptr(),
                                                      mu.data_ptr(), s_sum.data_ptr(), sn, monitor.data_ptr()),
               "gvq_compress_aggregate_monitored")

    def compress_quantize_aggregate(self, g_nodes, Ut, mu, levels, seed, s_sum, q_nodes=None, norms_nodes=None):
        self._sync_stream()
        qp = _ptr_array(q_nodes) if q_nodes is not None else None
        npp = _ptr_array(norms_nodes) if norms_nodes is not None else None
        _check(lib().gvq_compress_quantize_aggregate(self._h, _ptr_array(g_nodes), len(g_nodes), Ut.data_ptr(),
                                                     mu.data_ptr(), levels, seed, s_sum.data_ptr(), qp, npp),
               "gvq_compress_quantize_aggregate")

    def decompress(self, s_sum, Ut, mu, g_nodes_for_tails, N, g_hat):
        self._sync_stream()
        gp = _ptr_array(g_nodes_for_tails) if g_nodes_for_tails is not None else None
        _check(lib().gvq_decompress(self._h, s_sum.data_ptr(), Ut.data_ptr(), mu.data_ptr(), gp, N,
                                    g_hat.data_ptr()), "gvq_decompress")

    def fit_basis(self, hist, N, samples_are_sums_of, Ut, mu, evals):
        """Returns the per-layer sweep counts (host list)."""
        self._sync_stream()
        L = hist.shape[0]
        self.ensure_workspace(self.layout.fit_workspace_bytes(L))
        info = (ctypes.c_int32 * self.n_layers)()
        st = lib().gvq_fit_basis(self._h, hist.data_ptr(), hist.stride(0) if L > 1 else hist.shape[1], L, N,
                                 samples_are_sums_of, Ut.data_ptr(), mu.data_ptr(), evals.data_ptr(), info)
        _check(st, "gvq_fit_basis")
        return list(info)

    def fit_centre(self, hist, centre):
        """gvq_fit_centre: the point per layer that a fit spread over participants centres by."""
        self._sync_stream()
        L = hist.shape[0]
        _check(lib().gvq_fit_centre(self._h, hist.data_ptr(), hist.stride(0) if L > 1 else hist.shape[1], L,
                                    centre.data_ptr()), "gvq_fit_centre")

    def fit_moments(self, hist, centre, moments):
        """gvq_fit_moments: this participant's additive moments (fp64 [fit_moments_count]) about `centre`."""
        self._sync_stream()
        L = hist.shape[0]
        self.ensure_workspace(self.layout.fit_workspace_bytes(L))
        _check(lib().gvq_fit_moments(self._h, hist.data_ptr(), hist.stride(0) if L > 1 else hist.shape[1], L,
                                     centre.data_ptr(), moments.data_ptr()), "gvq_fit_moments")

    def fit_from_moments(self, moments, centre, N, samples_are_sums_of, Ut, mu, evals):
        """gvq_fit_from_moments: the fit from the summed moments.  Returns the per-layer sweep counts."""
        self._sync_stream()
        self.ensure_workspace(self.layout.fit_workspace_bytes(1))
        info = (ctypes.c_int32 * self.n_layers)()
        _check(lib().gvq_fit_from_moments(self._h, moments.data_ptr(), centre.data_ptr(), N, samples_are_sums_of,
                                          Ut.data_ptr(), mu.data_ptr(), evals.data_ptr(), info), "gvq_fit_from_moments")
        return list(info)

    def refresh_basis(self, hist, N, samples_are_sums_of, Ut, mu, evals_k, trace, iters=6, warm_start=True):
        """gvq_refresh_basis: the k leading eigenpairs by subspace iteration (Ut is read when warm_start)."""
        self._sync_stream()
        L = hist.shape[0]
        self.ensure_workspace(self.layout.fit_workspace_bytes(L))
        st = lib().gvq_refresh_basis(self._h, hist.data_ptr(), hist.stride(0) if L > 1 else hist.shape[1], L, N,
                                     samples_are_sums_of, 1 if warm_start else 0, iters, Ut.data_ptr(), mu.data_ptr(),
                                     evals_k.data_ptr(), trace.data_ptr())
        _check(st, "gvq_refresh_basis")

    def fit_basis_static(self, hist, N, samples_are_sums_of, Ut, mu, evals):
        """gvq_fit_basis_static: the same fit, with the library's built-in scratch array instead of a
        workspace -- for callers that cannot allocate device memory.  Returns the sweep counts."""
        self._sync_stream()
        L = hist.shape[0]
        info = (ctypes.c_int32 * self.n_layers)()
        st = lib().gvq_fit_basis_static(self._h, hist.data_ptr(), hist.stride(0) if L > 1 else hist.shape[1], L, N,
                                        samples_are_sums_of, Ut.data_ptr(), mu.data_ptr(), evals.data_ptr(), info)
        _check(st, "gvq_fit_basis_static")
        return list(info)

    def quantize(self, s_node, levels, seed, node, q, norms):
        self._sync_stream()
        _check(lib().gvq_quantize(self._h, s_node.data_ptr(), levels, seed, node, q.data_ptr(), norms.data_ptr()),
               "gvq_quantize")

    def quantize_aggregate(self, s_nodes, levels, seed, s_sum, q_nodes=None, norms_nodes=None):
        self._sync_stream()
        qp = _ptr_array(q_nodes) if q_nodes is not None else None
        npp = _ptr_array(norms_nodes) if norms_nodes is not None else None
        _check(lib().gvq_quantize_aggregate(self._h, _ptr_array(s_nodes), len(s_nodes), levels, seed, s_sum.data_ptr(),
                                            qp, npp), "gvq_quantize_aggregate")

    def dequantize_aggregate(self, q_nodes, norms_nodes, levels, s_sum):
        self._sync_stream()
        _check(lib().gvq_dequantize_aggregate(self._h, _ptr_array(q_nodes), _ptr_array(norms_nodes), levels,
                                              len(q_nodes), s_sum.data_ptr()), "gvq_dequantize_aggregate")

    def host_prepare(self):
        """gvq_host_prepare: builds the chunk pipeline of allreduce_host once (outside the training loop)."""
        _check(lib().gvq_host_prepare(self._h), "gvq_host_prepare")

    def allreduce_host(self, g_nodes_host, Ut, mu, g_hat_host, levels: int = 0, seed: int = 0):
        """g_nodes_host: CPU tensors (pinned for speed); Ut, mu: device; g_hat_host: CPU tensor.
        levels > 0: gvq_allreduce_host_quantized."""
        self._sync_stream()
        self.ensure_workspace(self.layout.host_workspace_bytes(len(g_nodes_host)))
        if levels > 0:
            _check(lib().gvq_allreduce_host_quantized(self._h, _ptr_array(g_nodes_host), len(g_nodes_host), Ut.data_ptr(),
                                                      mu.data_ptr(), levels, seed, g_hat_host.data_ptr()),
                   "gvq_allreduce_host_quantized")
        else:
            _check(lib().gvq_allreduce_host(self._h, _ptr_array(g_nodes_host), len(g_nodes_host), Ut.data_ptr(),
                                            mu.data_ptr(), g_hat_host.data_ptr()), "gvq_allreduce_host")
