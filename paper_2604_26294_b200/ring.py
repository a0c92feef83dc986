"""Algorithm 2 across real ranks: one process per GPU, each owning one token shard and one weight shard.

The single-GPU entry points keep all D shards resident, so nothing moves.  Here the shards really travel:
at every ring step a rank posts "send my current shard to p+1, receive the next one from p-1"
(AsyncRingSendRecv), computes the step with the shard it holds (`tsp_mlp_ring_step*`), waits, and swaps
buffers.  `torch.distributed` does the transport (NCCL over NVLink on GPUs; gloo on CPU, which is how the
schedule is tested without GPUs); every FLOP of a step runs in the library's kernels.

Backward pass: the weights travel as in the forward pass (Section 4.3.4: the backward mirrors the forward
weight movement) and the partial weight gradients are summed to the owner (Section 4.7) by an fp32
accumulator that travels WITH its shard: the rank holding shard k at step t adds its contribution and passes
the accumulator on, so after the last hop the owner holds the sum over the ranks in the order the shard met
them, r = (k + t) mod D.  This is a ring reduce-scatter whose transfers overlap the next step's GEMMs.

The two schedule functions are transport- and device-agnostic (compute is a callback); `TspRingMlp` binds them
to the CUDA library.
"""
from __future__ import annotations

import contextlib
from typing import Callable, Sequence

import torch
import torch.distributed as dist


def ring_neighbours(rank: int, D: int) -> tuple[int, int]:
    """(destination, source) of a rank's ring transfers: send to p+1, receive from p-1 (Algorithm 2)."""
    return (rank + 1) % D, (rank - 1) % D


def shard_at_step(rank: int, t: int, D: int) -> int:
    """Index of the weight shard rank `rank` holds at ring step t."""
    return (rank - t) % D


class DistTransport:
    """Ring transfers over torch.distributed (NCCL on GPUs, gloo on CPU): exchange() posts "send to p+1, receive from
    p-1" and returns requests with a wait() method."""

    def __init__(self, rank: int, D: int, group=None):
        dst, src = ring_neighbours(rank, D)
        if group is not None:
            dst, src = dist.get_global_rank(group, dst), dist.get_global_rank(group, src)
        self.dst, self.src, self.group = dst, src, group

    def exchange(self, send: torch.Tensor, recv: torch.Tensor):
        ops = [dist.P2POp(dist.isend, send, self.dst, self.group), dist.P2POp(dist.irecv, recv, self.src, self.group)]
        return dist.batch_isend_irecv(ops)


class HostOrder:
    """Ordering between transfers and compute when request.wait() blocks the host (gloo, CPU tensors): program order
    is enough, nothing to do."""

    def begin(self) -> None:                      # start of a pass, after the own shard has been copied into its row
        pass

    def end(self) -> None:                        # end of a pass, after the last transfer has been waited for
        pass

    def transport(self):
        return contextlib.nullcontext()

    def shard_arrived(self, t: int) -> None:      # called in the transport context right after the wait for shard t
        pass

    def before_compute(self, steps) -> None:      # called before the compute call that reads the shards of `steps`
        pass

    def after_compute(self, steps) -> None:       # called after that compute call has been issued
        pass

    def before_overwrite(self, t: int) -> None:   # called in the transport context before the buffer of step t is reused
        pass


class StreamOrder(HostOrder):
    """The same ordering on a GPU, where compute and transfers are asynchronous: every transfer is posted, and every
    request waited for, with a dedicated transport stream current (request.wait() of NCCL makes the CURRENT stream wait,
    so the compute stream is never held up by a transfer it does not need yet); the dependencies are explicit events:
      shard t has arrived          -> recorded on the transport stream, the compute stream waits for it before the
                                      compute call that reads shard t;
      the steps of a call are done -> recorded on the compute stream, the transport stream waits for it before a
                                      receive overwrites a buffer those steps read.
    Nothing here relies on how the transport orders consecutive transfers among themselves.
    """

    def __init__(self, device=None):
        self.compute = torch.cuda.current_stream(device)
        self.stream = torch.cuda.Stream(device=device)
        self.arrived: dict[int, torch.cuda.Event] = {}
        self.computed: dict[int, torch.cuda.Event] = {}

    def begin(self) -> None:
        """Start of a pass: transfers may read buffers the compute stream has just written (the own shard)."""
        self.compute = torch.cuda.current_stream()
        self.arrived.clear()
        self.computed.clear()
        self.stream.wait_stream(self.compute)

    def end(self) -> None:
        """End of a pass: later work on the compute stream comes after the last transfers."""
        self.compute.wait_stream(self.stream)

    def transport(self):
        return torch.cuda.stream(self.stream)

    def shard_arrived(self, t: int) -> None:
        ev = torch.cuda.Event()
        ev.record(self.stream)
        self.arrived[t] = ev

    def before_compute(self, steps) -> None:
        for t in steps:
            ev = self.arrived.pop(t, None)
            if ev is not None:
                self.compute.wait_event(ev)

    def after_compute(self, steps) -> None:
        ev = torch.cuda.Event()
        ev.record(self.compute)
        for t in steps:
            self.computed[t] = ev

    def before_overwrite(self, t: int) -> None:
        ev = self.computed.pop(t, None)
        if ev is not None:
            self.stream.wait_event(ev)


def _wait(reqs) -> None:
    for r in reqs:
        r.wait()


def ring_forward(compute: Callable[[int, int, torch.Tensor], None], own_shard: torch.Tensor,
                 recv_bufs: Sequence[torch.Tensor], rank: int, D: int, group=None,
                 before_exchange: Callable[[int], None] | None = None, transport=None) -> None:
    """The loop of Algorithm 2 on one rank.

    compute(t, k, shard) runs ring step t with the packed shard k = (rank - t) mod D it is handed;
    own_shard is this rank's packed shard (never written); recv_bufs are n >= 2 buffers of the same shape that
    take turns as receive target (step t receives into buffer t mod n, which step t - n + 1 was the last to read).
    The transfer for step t+1 is posted before step t computes.  before_exchange(t), if given, runs before the
    transfer of step t is posted: a caller whose compute is asynchronous uses it to make sure the target buffer's
    last reader has finished.
    """
    n = len(recv_bufs)
    cur = own_shard
    transport = transport or DistTransport(rank, D, group)
    for t in range(D):
        reqs = []
        if t < D - 1:
            if before_exchange is not None:
                before_exchange(t)
            nxt = recv_bufs[t % n]
            reqs = transport.exchange(cur, nxt)
        compute(t, shard_at_step(rank, t, D), cur)
        _wait(reqs)                      # Wait(): the next shard has arrived, the current one has left
        if t < D - 1:
            cur = nxt


def ring_forward_grouped(compute: Callable[[int, int, int], None], own_shard: torch.Tensor, slots: torch.Tensor,
                         rank: int, D: int, g: int, group=None, transport=None, order: HostOrder | None = None) -> None:
    """Algorithm 2 with g ring steps per compute call.

    With few tokens per rank one ring step does not fill a GPU, so a rank lets the transfers run ahead and applies
    g shards at a time.  slots [2g, n] is a ring of packed-shard buffers: the shard of step t lives in row t mod 2g,
    so the g shards of a group are consecutive rows (what `tsp_mlp_ring_steps` wants).  The rank's own shard is
    copied into row 0.  Every rank still forwards each shard it receives to p+1 exactly once: transfer t sends row
    (t-1) mod 2g and receives row t mod 2g, and is posted only after the receive of row (t-1) mod 2g has been waited
    for.  Before group j computes, the transfers for groups j and j+1 are posted, so the next group's shards arrive
    while this one computes.
    compute(t_first, n_steps, first_row) applies steps t_first .. t_first + n_steps - 1, whose shards are rows
    first_row .. first_row + n_steps - 1.
    transport: object with exchange(send, recv) -> requests (default: torch.distributed send / receive to the ring
    neighbours).  order: HostOrder (default; waits block the host) or StreamOrder (GPU: waits are stream-level, on a
    dedicated transport stream, with explicit events towards the compute stream).
    """
    pipe = _ShardPipeline(own_shard, slots, rank, D, g, transport or DistTransport(rank, D, group), order or HostOrder())
    for t0 in range(0, D, g):
        n = min(g, D - t0)
        pipe.fetch_group(t0, n)
        compute(t0, n, t0 % pipe.n_slots)
        pipe.group_issued(t0, n)
    pipe.finish()


class _ShardPipeline:
    """The weight shards of a rank running ahead of its compute through a ring of 2g packed buffers (see
    ring_forward_grouped): transfer t sends row (t-1) mod 2g to p+1 and receives the shard of step t into row t mod 2g."""

    def __init__(self, own_shard, slots, rank, D, g, transport, order):
        self.slots, self.rank, self.D, self.g = slots, rank, D, g
        self.transport, self.order = transport, order
        self.n_slots = slots.shape[0]
        assert self.n_slots >= 2 * g and g >= 1
        slots[0].copy_(own_shard)
        order.begin()
        self.reqs: dict[int, list] = {}               # transfer t -> its requests, until they have been waited for
        self.posted = 0                               # transfers 1 .. posted have been posted

    def _arrive(self, t: int) -> None:
        """Wait (once) for transfer t: shard t is in its row, and row (t-1) has been sent on."""
        if t in self.reqs:
            with self.order.transport():
                _wait(self.reqs.pop(t))
                self.order.shard_arrived(t)

    def _post_up_to(self, t_last: int) -> None:
        while self.posted < min(t_last, self.D - 1):
            t = self.posted + 1                       # delivers the shard of step t
            self._arrive(t - 1)                       # the shard about to be forwarded has arrived
            with self.order.transport():
                self.order.before_overwrite(t - self.n_slots)   # the steps that read row t mod 2g before are done
                self.reqs[t] = self.transport.exchange(self.slots[(t - 1) % self.n_slots], self.slots[t % self.n_slots])
            self.posted = t

    def fetch_group(self, t0: int, n: int) -> None:
        """Post the transfers of this group and the next, then wait for this group's shards."""
        self._post_up_to(t0 + n - 1 + self.g)
        for t in range(t0, t0 + n):
            self._arrive(t)
        self.order.before_compute(range(t0, t0 + n))

    def group_issued(self, t0: int, n: int) -> None:
        self.order.after_compute(range(t0, t0 + n))

    def finish(self) -> None:
        for t in sorted(self.reqs):                   # sends of the last transfers
            self._arrive(t)
        self.order.end()


def ring_backward(compute_dx: Callable[[int, int, torch.Tensor], None],
                  compute_dw: Callable[[int, int, torch.Tensor, bool], None], own_shard: torch.Tensor,
                  recv_bufs: Sequence[torch.Tensor], dw_bufs: Sequence[torch.Tensor], rank: int, D: int,
                  group=None, transport=None) -> torch.Tensor:
    """Backward ring on one rank; returns the buffer holding the summed gradient of this rank's OWN shard.

    compute_dx(t, k, shard): everything of step t that does not touch the weight-gradient accumulator.
    compute_dw(t, k, acc, accumulate): add (or, at t = 0, write) this rank's contribution for shard k into acc.
    dw_bufs: two fp32 buffers shaped like a packed shard; they alternate as "accumulator of the shard I hold"
    and "accumulator arriving for the next step".
    """
    cur = own_shard
    acc_reqs = []
    transport = transport or DistTransport(rank, D, group)
    for t in range(D):
        reqs = []
        if t < D - 1:
            nxt = recv_bufs[t & 1]
            reqs = transport.exchange(cur, nxt)
        k = shard_at_step(rank, t, D)
        compute_dx(t, k, cur)
        _wait(acc_reqs)                  # the accumulator of shard k has arrived from p-1 (nothing to wait for at t = 0)
        acc = dw_bufs[t & 1]
        compute_dw(t, k, acc, t > 0)
        if D > 1:                        # pass it on; the hop after the last step delivers it to the owner
            acc_reqs = transport.exchange(acc, dw_bufs[(t + 1) & 1])
        _wait(reqs)
        if t < D - 1:
            cur = nxt
    _wait(acc_reqs)
    return dw_bufs[D & 1] if D > 1 else dw_bufs[0]


def ring_backward_grouped(compute_group_dx: Callable[[int, int, int], None],
                          compute_dw: Callable[[int, int, int, torch.Tensor, bool], None], own_shard: torch.Tensor,
                          slots: torch.Tensor, dw_bufs: Sequence[torch.Tensor], rank: int, D: int, g: int, group=None,
                          transport=None, order: HostOrder | None = None) -> torch.Tensor:
    """Backward ring with g ring steps per compute call; returns the buffer holding the gradient of the rank's own shard.

    The weights run ahead exactly as in ring_forward_grouped (slots [2g, n]).  Per group of steps t_first .. t_first + n - 1
    compute_group_dx(t_first, n, first_row) does everything that does not touch a weight-gradient accumulator (dA, the
    recomputed gate|up GEMM with its backward epilogue for all n shards, the carried dX sum).  The accumulators keep
    travelling one shard at a time, because the accumulator of step t's shard leaves the left neighbour only after that
    rank has added its share: for every step of the group, in order, the rank waits for the accumulator, lets
    compute_dw(t, i, n, acc, accumulate) add the contribution of shard i of the group (at t = 0: write it), and passes
    it on.  The sum over ranks therefore runs in the order the shard meets them, r = (k + t) mod D, as in ring_backward,
    and only the kernels that do not depend on a neighbour's result are grouped.  The accumulator transfers are posted
    and waited for with the compute stream current: each depends on the kernel that has just written the accumulator.
    """
    transport = transport or DistTransport(rank, D, group)
    pipe = _ShardPipeline(own_shard, slots, rank, D, g, transport, order or HostOrder())
    acc_reqs = []
    for t0 in range(0, D, g):
        n = min(g, D - t0)
        pipe.fetch_group(t0, n)
        compute_group_dx(t0, n, t0 % pipe.n_slots)
        pipe.group_issued(t0, n)
        for i in range(n):
            t = t0 + i
            _wait(acc_reqs)              # the accumulator of this step's shard has arrived from p-1 (nothing at t = 0)
            acc = dw_bufs[t & 1]
            compute_dw(t, i, n, acc, t > 0)
            if D > 1:                    # pass it on; the hop after the last step delivers it to the owner
                acc_reqs = transport.exchange(acc, dw_bufs[(t + 1) & 1])
    pipe.finish()
    _wait(acc_reqs)
    return dw_bufs[D & 1] if D > 1 else dw_bufs[0]


def pack_shard(Wg_k: torch.Tensor, Wu_k: torch.Tensor, Wd_k: torch.Tensor) -> torch.Tensor:
    """One contiguous message per ring step: [Wg_k | Wu_k | Wd_k] flattened."""
    return torch.cat([Wg_k.reshape(-1), Wu_k.reshape(-1), Wd_k.reshape(-1)])


def unpack_shard(buf: torch.Tensor, H: int, F_d: int):
    """Views (Wg_k [H, F_d], Wu_k [H, F_d], Wd_k [F_d, H]) into a packed shard (or packed gradient) buffer."""
    n = H * F_d
    return buf[:n].view(H, F_d), buf[n:2 * n].view(H, F_d), buf[2 * n:3 * n].view(F_d, H)


class TspRingMlp:
    """One rank of the TSP gated ring MLP on its own GPU: the schedule above driving the library's step kernels."""

    # up to this many tokens per rank the two halves of a forward step run on two streams (measured on one rank's
    # step sequence: +3 % at 1024 tokens, +6 % at 2048, -2 % at 8192)
    TWO_STREAM_MAX_TOKENS = 4096

    def __init__(self, H: int, F: int, D: int, rank: int, S_loc: int, group=None, training: bool = False,
                 activation: int | None = None, steps_per_launch: int | None = None):
        from . import binding as b   # fails loudly without the CUDA library or a GPU

        self.b, self.H, self.F, self.D, self.rank, self.S_loc, self.group = b, H, F, D, rank, S_loc, group
        self.F_d = F // D
        dev = torch.device("cuda", torch.cuda.current_device())
        self.plan = b.tsp_mlp_plan(H, F, D)
        if activation is not None:
            b.tsp_mlp_set_activation(self.plan, activation)
        # ring steps applied per group of launches, forward and backward (measured on one rank's step sequence at
        # H = 4096, F/D = 1792, forward: 1024 tokens per rank 1027 -> 1215 / 1305 TFLOP/s with 2 / 4 steps per launch; 8192
        # tokens 1277 -> 1452 / 1505); more steps per launch also mean more shards in flight (2 g receive buffers)
        if steps_per_launch is None:
            steps_per_launch = 4 if S_loc <= 2048 else 2
        self.g = max(1, min(steps_per_launch, D))
        nbytes = max(b.tsp_mlp_workspace_bytes_ring(self.plan, S_loc, b.TSP_WS_BACKWARD if training else b.TSP_WS_FORWARD),
                     b.tsp_mlp_workspace_bytes_ring_group(self.plan, S_loc, self.g),
                     b.tsp_mlp_workspace_bytes_ring_group_backward(self.plan, S_loc, self.g) if training else 0)
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        b.tsp_mlp_set_workspace(self.plan, self.workspace)
        n = 3 * H * self.F_d
        # three receive buffers: the down projection of step t may still read its shard while the transfer for
        # step t+2 is posted (the two halves of a step run on two streams, see forward())
        self.recv_bufs = [torch.empty(n, dtype=torch.bfloat16, device=dev) for _ in range(3)] if D > 1 else []
        self.dw_bufs = [torch.empty(n, dtype=torch.float32, device=dev) for _ in range(2 if D > 1 else 1)] if training else []
        self.slots = torch.empty(2 * self.g, n, dtype=torch.bfloat16, device=dev) if (D > 1 and self.g > 1) else None
        self.down_stream = torch.cuda.Stream(device=dev)
        self.order = StreamOrder(dev)                 # transfers of the grouped schedules: own stream, explicit events
        self._gate_done = [torch.cuda.Event() for _ in range(D)]
        self._down_done = [torch.cuda.Event() for _ in range(D)]

    def close(self) -> None:
        if self.plan is not None:
            self.b.tsp_mlp_plan_destroy(self.plan)
            self.plan = None

    def forward(self, X_p: torch.Tensor, shard: torch.Tensor, Y_p: torch.Tensor | None = None) -> torch.Tensor:
        """Y_p = rows of this rank of the gated MLP over all D shards; `shard` is this rank's packed own shard.

        The gate|up GEMM of step t runs on the current stream, the down projection of step t on a second stream, so
        that the down projection overlaps the next step's gate|up GEMM (with few tokens per rank neither fills the
        GPU alone; with many tokens per rank everything stays on the current stream).  On return the current stream
        has been made to wait for the last down projection.
        """
        if Y_p is None:
            Y_p = torch.empty_like(X_p)
        main = torch.cuda.current_stream()
        if self.slots is not None:                    # g ring steps per launch
            n = 3 * self.H * self.F_d

            def compute_group(t_first, n_steps, first_row):
                Wg, Wu, Wd = unpack_shard(self.slots[first_row], self.H, self.F_d)
                self.b.tsp_mlp_ring_steps(self.plan, X_p, Wg, Wu, Wd, n, n_steps, Y_p, self.S_loc, t_first, self.D, main)

            ring_forward_grouped(compute_group, shard, self.slots, self.rank, self.D, self.g, self.group,
                                 order=self.order)
            return Y_p
        if self.S_loc > self.TWO_STREAM_MAX_TOKENS:   # a step fills the GPU by itself: one stream, no event traffic
            def compute_one_stream(t, k, buf):
                Wg, Wu, Wd = unpack_shard(buf, self.H, self.F_d)
                self.b.tsp_mlp_ring_step(self.plan, X_p, Wg, Wu, Wd, Y_p, self.S_loc, t, self.D, main)

            ring_forward(compute_one_stream, shard, self.recv_bufs, self.rank, self.D, self.group)
            return Y_p
        self.down_stream.wait_stream(main)            # whatever produced X_p, shard and freed Y_p comes first

        def before_exchange(t):
            if t >= 2:                                # the receive buffer of step t was last read by step t - 2
                main.wait_event(self._down_done[t - 2])

        def compute(t, k, buf):
            Wg, Wu, Wd = unpack_shard(buf, self.H, self.F_d)
            if t >= 2:                                # scratch buffer t & 1 is free once down(t - 2) has run
                main.wait_event(self._down_done[t - 2])
            self.b.tsp_mlp_ring_step_gate(self.plan, X_p, Wg, Wu, self.S_loc, t, self.D, main)
            self._gate_done[t].record(main)
            self.down_stream.wait_event(self._gate_done[t])
            self.b.tsp_mlp_ring_step_down(self.plan, Wd, Y_p, self.S_loc, t, self.D, self.down_stream)
            self._down_done[t].record(self.down_stream)

        ring_forward(compute, shard, self.recv_bufs, self.rank, self.D, self.group, before_exchange)
        main.wait_stream(self.down_stream)
        return Y_p

    def backward(self, X_p: torch.Tensor, shard: torch.Tensor, dY_p: torch.Tensor, dX_p: torch.Tensor | None = None):
        """Returns (dX_p, (dWg, dWu, dWd)) with the weight gradients of this rank's own shard, fp32, summed over ranks."""
        if not self.dw_bufs:
            raise RuntimeError("TspRingMlp was created with training=False")
        if dX_p is None:
            dX_p = torch.empty_like(X_p)

        if self.slots is not None:                    # g ring steps per launch group; accumulators still one by one
            n_elems = 3 * self.H * self.F_d

            def compute_group_dx(t_first, n_steps, first_row):
                Wg, Wu, Wd = unpack_shard(self.slots[first_row], self.H, self.F_d)
                self.b.tsp_mlp_ring_steps_backward_dx(self.plan, X_p, Wg, Wu, Wd, n_elems, n_steps, dY_p, dX_p, self.S_loc,
                                                      t_first, self.D)

            def compute_dw_of_group(t, i, n_steps, acc, accumulate):
                dWg, dWu, dWd = unpack_shard(acc, self.H, self.F_d)
                self.b.tsp_mlp_ring_steps_backward_dw(self.plan, X_p, dY_p, dWg, dWu, dWd, self.S_loc, i, n_steps,
                                                      int(accumulate), self.D)

            out = ring_backward_grouped(compute_group_dx, compute_dw_of_group, shard, self.slots, self.dw_bufs, self.rank,
                                        self.D, self.g, self.group, order=self.order)
            return dX_p, unpack_shard(out, self.H, self.F_d)

        def compute_dx(t, k, buf):
            Wg, Wu, Wd = unpack_shard(buf, self.H, self.F_d)
            self.b.tsp_mlp_ring_step_backward_dx(self.plan, X_p, Wg, Wu, Wd, dY_p, dX_p, self.S_loc, t, self.D)

        def compute_dw(t, k, acc, accumulate):
            dWg, dWu, dWd = unpack_shard(acc, self.H, self.F_d)
            self.b.tsp_mlp_ring_step_backward_dw(self.plan, X_p, dY_p, dWg, dWu, dWd, self.S_loc, int(accumulate), self.D)

        out = ring_backward(compute_dx, compute_dw, shard, self.recv_bufs, self.dw_bufs, self.rank, self.D, self.group)
        return dX_p, unpack_shard(out, self.H, self.F_d)
