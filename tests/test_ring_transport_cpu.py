"""The grouped ring schedules against an adversarial transport, on CPU, with the D ranks as threads.

The fake transport is as unhelpful as an asynchronous transport may be:
  * a send captures its buffer at the moment it is POSTED (so a shard forwarded before its own receive has been waited
    for travels on with stale contents), and
  * a receive writes its buffer only when its request is WAITED for (so a buffer read before the wait holds the previous
    contents), and a request may be waited for once only.
The schedules must reach the unsharded result under these rules; a deliberately broken variant (forwarding without
waiting) must not, which shows that the fake would notice.
"""
import threading

import numpy as np
import pytest
import torch

from oracle import tsp_mlp_oracle as orc
from paper_2604_26294_b200 import inputs as inp
from paper_2604_26294_b200 import ring


class _Request:
    def __init__(self, fn):
        self._fn = fn

    def wait(self):
        assert self._fn is not None, "a request was waited for twice"
        fn, self._fn = self._fn, None
        fn()


class _Edge:
    """Messages of one directed edge; receive number n (in posting order) gets message number n, whenever it is waited for."""

    def __init__(self):
        self.messages, self.cv = [], threading.Condition()

    def put(self, msg):
        with self.cv:
            self.messages.append(msg)
            self.cv.notify_all()

    def get(self, n):
        with self.cv:
            assert self.cv.wait_for(lambda: len(self.messages) > n, timeout=60), "message never sent"
            return self.messages[n]


class FakeTransport:
    """One rank's end of a ring of in-process mailboxes (one per directed edge)."""

    def __init__(self, rank, D, boxes):
        dst, src = ring.ring_neighbours(rank, D)
        self.out_box, self.in_box = boxes[(rank, dst)], boxes[(src, rank)]
        self.n_recv = 0

    def exchange(self, send, recv):
        self.out_box.put(send.clone())                       # captured when posted
        n, self.n_recv = self.n_recv, self.n_recv + 1        # matched in posting order, like a real transport

        def deliver():
            recv.copy_(self.in_box.get(n))                   # lands when waited for
        return [_Request(lambda: None), _Request(deliver)]


def _run_ranks(D, g, broken=False):
    S, H, F = 6 * D, 8, 4 * D
    S_loc, F_d = S // D, F // D
    host = inp.make_inputs(S, H, F, seed=9, with_dy=True)
    X, Wg, Wu, Wd, dY = (inp.bf16_bits_to_f64(a) for a in (host.X, host.Wg, host.Wu, host.Wd, host.dY))
    boxes = {(r, (r + 1) % D): _Edge() for r in range(D)}
    out, errors = {}, []

    def rank_main(rank):
        try:
            Xp, dYp = X[rank * S_loc:(rank + 1) * S_loc], dY[rank * S_loc:(rank + 1) * S_loc]
            cols = slice(rank * F_d, (rank + 1) * F_d)
            own = ring.pack_shard(torch.from_numpy(Wg[:, cols].copy()), torch.from_numpy(Wu[:, cols].copy()),
                                  torch.from_numpy(Wd[cols, :].copy()))
            slots = torch.full((2 * g, own.numel()), float("nan"), dtype=own.dtype)
            transport = FakeTransport(rank, D, boxes)
            Yp = np.zeros((S_loc, H))

            def compute(t_first, n, first_row):
                for i in range(n):
                    wg, wu, wd = (a.numpy() for a in ring.unpack_shard(slots[first_row + i], H, F_d))
                    Yp[...] += orc.gated_mlp_forward(Xp, wg, wu, wd)

            ring.ring_forward_grouped(compute, own, slots, rank, D, g, transport=transport)

            dXp, parts = np.zeros((S_loc, H)), {}

            def compute_group_dx(t_first, n, first_row):
                for i in range(n):
                    wg, wu, wd = (a.numpy() for a in ring.unpack_shard(slots[first_row + i], H, F_d))
                    dx, dwg, dwu, dwd = orc.gated_mlp_backward(Xp, wg, wu, wd, dYp)
                    dXp[...] += dx
                    parts[i] = ring.pack_shard(torch.from_numpy(dwg), torch.from_numpy(dwu), torch.from_numpy(dwd))

            def compute_dw(t, i, n, acc, accumulate):
                if accumulate:
                    acc += parts[i]
                else:
                    acc.copy_(parts[i])

            slots.fill_(float("nan"))
            dw_bufs = [torch.full_like(own, float("nan")) for _ in range(2)]
            mine = ring.ring_backward_grouped(compute_group_dx, compute_dw, own, slots, dw_bufs, rank, D, g,
                                              transport=transport)
            out[rank] = (Yp, dXp, [a.numpy().copy() for a in ring.unpack_shard(mine, H, F_d)])
        except Exception as e:   # noqa: BLE001 - reported by the main thread
            errors.append((rank, repr(e)))

    saved = ring._ShardPipeline._arrive
    if broken:   # forward shards without waiting for them first (what an implicit ordering assumption would do)
        def lazy_arrive(self, t, _orig=saved):
            if getattr(self, "_fetching", False):
                _orig(self, t)
        def fetch(self, t0, n, _orig=ring._ShardPipeline.fetch_group):
            self._post_up_to(t0 + n - 1 + self.g)
            self._fetching = True
            for t in range(t0, t0 + n):
                self._arrive(t)
            self._fetching = False
        ring._ShardPipeline._arrive, saved_fetch = lazy_arrive, ring._ShardPipeline.fetch_group
        ring._ShardPipeline.fetch_group = fetch
    try:
        threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(D)]
        for t in threads:
            t.start()
        for t in threads:
            t.join(120)
    finally:
        ring._ShardPipeline._arrive = saved
        if broken:
            ring._ShardPipeline.fetch_group = saved_fetch
    Y_ref = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    worst = 0.0
    for r in range(D):
        if r not in out:
            return float("inf"), errors
        rows, cols = slice(r * S_loc, (r + 1) * S_loc), slice(r * F_d, (r + 1) * F_d)
        Yp, dXp, (dWg, dWu, dWd) = out[r]
        for got, ref in ((Yp, Y_ref[rows]), (dXp, rdX[rows]), (dWg, rdWg[:, cols]), (dWu, rdWu[:, cols]),
                         (dWd, rdWd[cols, :])):
            diff = np.abs(got - ref)
            worst = max(worst, float(np.max(np.where(np.isfinite(diff), diff, np.inf)) / np.max(np.abs(ref))))
    return worst, errors


@pytest.mark.parametrize("D,g", [(2, 2), (3, 2), (4, 2), (5, 2), (5, 3), (8, 4), (4, 1)])
def test_grouped_schedules_wait_before_they_forward(D, g):
    worst, errors = _run_ranks(D, g)
    assert not errors, errors
    assert worst <= 1e-12, worst


def test_the_fake_transport_notices_a_missing_wait():
    worst, errors = _run_ranks(4, 2, broken=True)
    assert errors or not worst <= 1e-12      # stale shards travel on: a wrong (or non-finite) result, or a failed check
