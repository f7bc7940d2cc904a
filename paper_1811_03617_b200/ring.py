"""Algorithm 1 across processes: compressed-domain ring all-reduce, one segment per participant.

Plumbing only.  Every arithmetic step is a kernel behind the C ABI (``gvq_compress_aggregate_partial``,
``gvq_exchange_accumulate``, ``gvq_decompress_exchanged``), reached through a *segment engine*; the messages are
moved by a *transport* (``torch.distributed`` point-to-point operations, NCCL between GPUs).  A participant is one
process with one GPU that holds ``n_local >= 1`` of the job's N node gradients (the paper's setting is
n_local = 1).

The schedule is Algorithm 1's, with the send that closes step i - 1 posted together with the receive that opens
step i, so that both directions of a link are busy at once:

  compression round     step 0        x[n] = Q(g(n))
                        step i >= 1   send x[n - i + 1] on, receive r;  meanwhile x[n - i] = Q(g(n - i));
                                      then x[n - i] += r
  decompression round   step i        send x[n + 1 - i] on, receive x[n - i];  meanwhile decompress x[n + 1 - i]
                                      (the last step receives nothing)

Indices are modulo the ring size W; Q is Eq. 3 on the participant's own gradients with the mean scaled by 1 / N.
The transfer of a step overlaps that step's kernel: point-to-point operations run on the communication library's
own stream, which waits for the kernels enqueued before the operation was posted, and ``wait()`` makes the
compute stream wait for the transfer.

``post`` / ``finish`` halves of a step are separate methods so that several participants can be stepped in
lock-step inside one process (``LocalRing``): that is how a single GPU checks the schedule, the segment layouts
and the kernels against the oracle without kernels that wait on one another.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import gvq


# --------------------------------------------------------------------------------------- engine
class CudaSegmentEngine:
    """One gvq context per segment of the layout (gvq_segment_layout), all on one device."""

    def __init__(self, layout, n_segments: int, device: Optional[int] = None):
        self.layout = layout if isinstance(layout, gvq.HostLayout) else gvq.HostLayout.of(layout)
        self.n_segments = int(n_segments)
        self.device = torch.cuda.current_device() if device is None else int(device)
        self.ctx: List[Optional[gvq.Context]] = []
        self.layers: List[List[int]] = []
        self.x_floats: List[int] = []
        self._views = {}
        for j in range(self.n_segments):
            seg, layers = gvq.segment_layout(self.layout, self.n_segments, j)
            self.ctx.append(None if seg is None else gvq.Context(seg, self.device))
            self.layers.append(layers)
            self.x_floats.append(0 if seg is None else seg.exchange_floats())

    def new_buffer(self, n_floats: int) -> torch.Tensor:
        return torch.empty(max(n_floats, 4), dtype=torch.float32, device=f"cuda:{self.device}")

    def _basis(self, j, Ut, mu):
        """Rows of (Ut, mu) of the layers that segment j's pieces were cut from."""
        ls = self.layers[j]
        if ls[-1] - ls[0] + 1 == len(ls):          # consecutive layers: views, no copy (kept per buffer)
            key = (j, Ut.data_ptr(), mu.data_ptr())
            hit = self._views.get(key)
            if hit is None:
                if len(self._views) > 4 * self.n_segments:
                    self._views.clear()
                hit = self._views[key] = (Ut[ls[0]:ls[-1] + 1], mu[ls[0]:ls[-1] + 1])
            return hit
        idx = torch.tensor(ls, device=Ut.device)   # pieces skip an empty layer: gather (the values may have changed)
        return Ut.index_select(0, idx).contiguous(), mu.index_select(0, idx).contiguous()

    def compress(self, j, g_local: Sequence[torch.Tensor], N: int, Ut, mu, x):
        if self.ctx[j] is not None:
            U, m = self._basis(j, Ut, mu)
            self.ctx[j].compress_aggregate_partial(g_local, N, U, m, x)

    def accumulate(self, j, x_acc, x_in):
        if self.ctx[j] is not None:
            self.ctx[j].exchange_accumulate(x_acc, x_in)

    def decompress(self, j, x, Ut, mu, g_hat):
        if self.ctx[j] is not None:
            U, m = self._basis(j, Ut, mu)
            self.ctx[j].decompress_exchanged(x, U, m, g_hat)

    def close(self):
        for c in self.ctx:
            if c is not None:
                c.close()


# ------------------------------------------------------------------------------------ transports
class _Done:
    def wait(self):
        return None


class DistTransport:
    """Successor / predecessor exchange over a torch.distributed process group (NCCL for GPU buffers)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.rank = dist.get_rank(group)
        self.world = dist.get_world_size(group)

    class _Reqs:
        def __init__(self, reqs):
            self.reqs = reqs

        def wait(self):
            for r in self.reqs:
                r.wait()

    def exchange(self, send: Optional[torch.Tensor], recv: Optional[torch.Tensor]):
        dist = self.dist
        if self.world == 1:
            return _Done()
        succ = dist.get_global_rank(self.group, (self.rank + 1) % self.world) if self.group is not None \
            else (self.rank + 1) % self.world
        pred = dist.get_global_rank(self.group, (self.rank - 1) % self.world) if self.group is not None \
            else (self.rank - 1) % self.world
        ops = []
        if send is not None and send.numel() > 0:
            ops.append(dist.P2POp(dist.isend, send, succ, self.group))
        if recv is not None and recv.numel() > 0:
            ops.append(dist.P2POp(dist.irecv, recv, pred, self.group))
        return self._Reqs(dist.batch_isend_irecv(ops)) if ops else _Done()


class _LocalLink:
    """The transport of one participant of a LocalRing: a receive copies what the predecessor posted."""

    def __init__(self, ring: "LocalRing", rank: int):
        self.ring, self.rank, self.world = ring, rank, ring.world
        self.posted: Optional[torch.Tensor] = None

    class _Copy:
        def __init__(self, link, recv):
            self.link, self.recv = link, recv

        def wait(self):
            if self.recv is not None and self.recv.numel() > 0:
                src = self.link.ring.links[(self.link.rank - 1) % self.link.world].posted
                self.recv.copy_(src)

    def exchange(self, send, recv):
        self.posted = send
        return self._Copy(self, recv)


# ---------------------------------------------------------------------------------- participant
class RingParticipant:
    """One node of Algorithm 1."""

    def __init__(self, engine, transport, rank: Optional[int] = None, world: Optional[int] = None):
        self.engine, self.transport = engine, transport
        self.rank = transport.rank if rank is None else rank
        self.world = transport.world if world is None else world
        if engine.n_segments != self.world:
            raise ValueError("Algorithm 1 uses one segment per participant")
        W = self.world
        self.x = [engine.new_buffer(engine.x_floats[j]) for j in range(W)]
        self.r = engine.new_buffer(max(engine.x_floats))
        self._pending = None
        self._xviews = {}
        self.floats_sent = 0

    def _view(self, buf, j):
        key = (buf.data_ptr(), j)
        v = self._xviews.get(key)
        if v is None:
            v = self._xviews[key] = buf[: self.engine.x_floats[j]]
        return v

    def begin(self, g_local: Sequence[torch.Tensor], N: int, Ut, mu, g_hat):
        self.g_local, self.N, self.Ut, self.mu, self.g_hat = list(g_local), int(N), Ut, mu, g_hat
        self.floats_sent = 0

    def _exchange(self, send_j: Optional[int], recv_buf, recv_j: Optional[int]):
        send = None if send_j is None else self._view(self.x[send_j], send_j)
        recv = None if recv_j is None else self._view(recv_buf, recv_j)
        if send is not None:
            self.floats_sent += send.numel()
        self._pending = self.transport.exchange(send, recv)

    # compression round ------------------------------------------------------------------
    def compress_post(self, i: int):
        n, W = self.rank, self.world
        j = (n - i) % W
        if i >= 1:
            self._exchange((n - i + 1) % W, self.r, j)
        self.engine.compress(j, self.g_local, self.N, self.Ut, self.mu, self.x[j])

    def compress_finish(self, i: int):
        if i >= 1:
            j = (self.rank - i) % self.world
            self._pending.wait()
            self.engine.accumulate(j, self._view(self.x[j], j), self._view(self.r, j))

    # decompression round ----------------------------------------------------------------
    def decompress_post(self, i: int):
        n, W = self.rank, self.world
        j = (n + 1 - i) % W
        if i < W - 1:
            self._exchange(j, self.x[(n - i) % W], (n - i) % W)
        else:
            self._pending = _Done()
        self.engine.decompress(j, self.x[j], self.Ut, self.mu, self.g_hat)

    def decompress_finish(self, i: int):
        self._pending.wait()

    def run(self, g_local, N, Ut, mu, g_hat):
        """The whole of Algorithm 1 for this participant; kernels and transfers are only enqueued."""
        self.begin(g_local, N, Ut, mu, g_hat)
        for i in range(self.world):
            self.compress_post(i)
            self.compress_finish(i)
        for i in range(self.world):
            self.decompress_post(i)
            self.decompress_finish(i)
        return g_hat


class LocalRing:
    """W participants of Algorithm 1 stepped in lock-step inside one process, buffers of all of them on the
    engine's device: the single-GPU form of the multi-process ring (same kernels, same schedule, copies in place
    of the link)."""

    def __init__(self, engine_factory, world: int):
        self.world = int(world)
        self.links = [_LocalLink(self, n) for n in range(self.world)]
        self.nodes = [RingParticipant(engine_factory(), self.links[n], n, self.world) for n in range(self.world)]

    def run(self, g_by_rank: Sequence[Sequence[torch.Tensor]], N: int, Ut, mu, g_hat_by_rank):
        for n, p in enumerate(self.nodes):
            p.begin(g_by_rank[n], N, Ut, mu, g_hat_by_rank[n])
        for i in range(self.world):
            for p in self.nodes:
                p.compress_post(i)
            for p in self.nodes:
                p.compress_finish(i)
        for i in range(self.world):
            for p in self.nodes:
                p.decompress_post(i)
            for p in self.nodes:
                p.decompress_finish(i)
        return g_hat_by_rank


# ------------------------------------------------------------------- library-collective variant
class _ContextEngine:
    """A gvq.Context over the whole layout seen as a segment engine with the single segment 0."""
    n_segments = 1

    def __init__(self, ctx: "gvq.Context"):
        self.ctx = ctx
        self.x_floats = [ctx.layout.exchange_floats()]

    def new_buffer(self, n_floats: int) -> torch.Tensor:
        return torch.empty(max(n_floats, 4), dtype=torch.float32, device=f"cuda:{self.ctx.device}")

    def compress(self, j, g_local, N, Ut, mu, x):
        self.ctx.compress_aggregate_partial(g_local, N, Ut, mu, x)

    def decompress(self, j, x, Ut, mu, g_hat):
        self.ctx.decompress_exchanged(x, Ut, mu, g_hat)

    def pack(self, x, x_packed):
        self.ctx.exchange_pack(x, x_packed)

    def unpack(self, x_packed, x):
        self.ctx.exchange_unpack(x_packed, x)


def allreduce_compressed(engine, g_local, N: int, Ut, mu, x, g_hat, group=None, x_packed=None):
    """Eq. 3 on the local gradients, ONE library all-reduce of the exchange buffer (k / d of the raw gradient's
    bytes; NCCL may reduce it inside the switch), Eq. 5.  The same result as the ring up to the summation order.
    engine: a segment engine whose single segment is the whole layout (CudaSegmentEngine(layout, 1)), or a
    gvq.Context over the whole layout.  x: an exchange buffer of engine.x_floats[0] floats (engine.new_buffer).
    x_packed: with per-layer compressed lengths (the basis masked, gvq_set_layer_k called on the context) a buffer
    of gvq_packed_floats() floats: the collective then carries only the coordinates that can be non-zero."""
    import torch.distributed as dist
    if isinstance(engine, gvq.Context):
        engine = _ContextEngine(engine)
    if engine.n_segments != 1:
        raise ValueError("the library-collective variant works on the whole layout: an engine with one segment")
    engine.compress(0, g_local, N, Ut, mu, x)
    many = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    if x_packed is not None:
        engine.pack(x, x_packed)
        if many:
            dist.all_reduce(x_packed, group=group)
        engine.unpack(x_packed, x)
    elif many:
        dist.all_reduce(x, group=group)
    engine.decompress(0, x, Ut, mu, g_hat)
    return g_hat
