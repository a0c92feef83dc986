"""Worker for tests/test_ring_schedule_cpu.py: one rank of a gloo group on CPU running the ring schedules.

The transport and the schedule are the product's (paper_2604_26294_b200/ring.py); the per-step arithmetic is
stood in for by the fp64 oracle on CPU tensors, so the test shows that every rank meets every shard exactly once,
in ring order, and that the travelling weight-gradient accumulators end up at their owners.
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402
import torch.distributed as dist  # noqa: E402

from oracle import tsp_mlp_oracle as orc  # noqa: E402
from paper_2604_26294_b200 import inputs as inp  # noqa: E402
from paper_2604_26294_b200 import ring  # noqa: E402


def main():
    out_dir = sys.argv[1]
    dist.init_process_group("gloo")
    rank, D = dist.get_rank(), dist.get_world_size()
    S, H, F = 12 * D, 8, 6 * D
    S_loc, F_d = S // D, F // D
    host = inp.make_inputs(S, H, F, seed=5, with_dy=True)      # every rank draws the same full problem ...
    X, Wg, Wu, Wd, dY = (inp.bf16_bits_to_f64(a) for a in (host.X, host.Wg, host.Wu, host.Wd, host.dY))
    Xp, dYp = X[rank * S_loc:(rank + 1) * S_loc], dY[rank * S_loc:(rank + 1) * S_loc]
    cols = slice(rank * F_d, (rank + 1) * F_d)                  # ... and keeps only its own shards
    own = ring.pack_shard(torch.from_numpy(Wg[:, cols].copy()), torch.from_numpy(Wu[:, cols].copy()),
                          torch.from_numpy(Wd[cols, :].copy()))
    recv = [torch.empty_like(own) for _ in range(3)]    # three take turns in the forward pass, the first two in the backward
    visited, hook_calls = [], []

    # ---- forward
    Yp = np.zeros((S_loc, H))

    def compute(t, k, buf):
        wg, wu, wd = (a.numpy() for a in ring.unpack_shard(buf, H, F_d))
        assert np.array_equal(wg, Wg[:, k * F_d:(k + 1) * F_d]), "the shard handed over is not shard k"
        visited.append(k)
        Yp[...] += orc.gated_mlp_forward(Xp, wg, wu, wd)

    ring.ring_forward(compute, own, recv, rank, D, before_exchange=hook_calls.append)

    # ---- forward again, two ring steps per compute call (the transfers run ahead through a ring of 4 buffers)
    Yg = np.zeros((S_loc, H))
    groups = []
    slots = torch.full((4, own.numel()), float("nan"), dtype=own.dtype)

    def compute_group(t_first, n_steps, first_row):
        groups.append((t_first, n_steps, first_row))
        for i in range(n_steps):
            k = ring.shard_at_step(rank, t_first + i, D)
            wg, wu, wd = (a.numpy() for a in ring.unpack_shard(slots[first_row + i], H, F_d))
            assert np.array_equal(wu, Wu[:, k * F_d:(k + 1) * F_d]), "row does not hold the shard of that step"
            Yg[...] += orc.gated_mlp_forward(Xp, wg, wu, wd)

    ring.ring_forward_grouped(compute_group, own, slots, rank, D, 2)

    # ---- backward
    dXp = np.zeros((S_loc, H))
    parts = {}

    def compute_dx(t, k, buf):
        wg, wu, wd = (a.numpy() for a in ring.unpack_shard(buf, H, F_d))
        assert np.array_equal(wd, Wd[k * F_d:(k + 1) * F_d, :])
        dx, dwg, dwu, dwd = orc.gated_mlp_backward(Xp, wg, wu, wd, dYp)
        dXp[...] += dx
        parts["dw"] = ring.pack_shard(torch.from_numpy(dwg), torch.from_numpy(dwu), torch.from_numpy(dwd))

    # every accumulator carries one extra element: the ranks that added to it, as base-D digits in visiting order
    def add_to(acc, part, accumulate):
        if accumulate:
            acc[:-1] += part
            acc[-1] = acc[-1] * D + rank
        else:
            acc[:-1].copy_(part)
            acc[-1] = rank

    def compute_dw(t, k, acc, accumulate):
        add_to(acc, parts["dw"], accumulate)

    n_acc = own.numel() + 1
    dw_bufs = [torch.full((n_acc,), float("nan"), dtype=own.dtype) for _ in range(2)]
    mine = ring.ring_backward(compute_dx, compute_dw, own, recv, dw_bufs, rank, D)
    trace = int(mine[-1].item())
    dWg_own, dWu_own, dWd_own = (a.numpy() for a in ring.unpack_shard(mine[:-1], H, F_d))

    # ---- backward again, two ring steps per compute call: only what does not depend on the left neighbour is grouped
    dXg = np.zeros((S_loc, H))
    gparts, bgroups = {}, []

    def compute_group_dx(t_first, n_steps, first_row):
        bgroups.append((t_first, n_steps, first_row))
        gparts.clear()
        for i in range(n_steps):
            k = ring.shard_at_step(rank, t_first + i, D)
            wg, wu, wd = (a.numpy() for a in ring.unpack_shard(slots[first_row + i], H, F_d))
            assert np.array_equal(wg, Wg[:, k * F_d:(k + 1) * F_d]), "row does not hold the shard of that step"
            dx, dwg, dwu, dwd = orc.gated_mlp_backward(Xp, wg, wu, wd, dYp)
            dXg[...] += dx
            gparts[i] = ring.pack_shard(torch.from_numpy(dwg), torch.from_numpy(dwu), torch.from_numpy(dwd))

    def compute_dw_of_group(t, i, n_steps, acc, accumulate):
        add_to(acc, gparts[i], accumulate)

    slots.fill_(float("nan"))
    dw_bufs = [torch.full((n_acc,), float("nan"), dtype=own.dtype) for _ in range(2)]
    mine_g = ring.ring_backward_grouped(compute_group_dx, compute_dw_of_group, own, slots, dw_bufs, rank, D, 2)
    trace_g = int(mine_g[-1].item())
    gWg, gWu, gWd = (a.numpy() for a in ring.unpack_shard(mine_g[:-1], H, F_d))

    # ---- compare with the unsharded definition
    Y_ref = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    rows = slice(rank * S_loc, (rank + 1) * S_loc)

    def err(a, ref):
        return float(np.max(np.abs(a - ref)) / np.max(np.abs(ref)))

    out = {"rank": rank, "D": D, "visited": visited, "hook_calls": hook_calls,
           "groups": groups, "err_Y_grouped": err(Yg, Y_ref[rows]),
           "err_Y": err(Yp, Y_ref[rows]), "err_dX": err(dXp, rdX[rows]),
           "err_dWg": err(dWg_own, rdWg[:, cols]), "err_dWu": err(dWu_own, rdWu[:, cols]),
           "err_dWd": err(dWd_own, rdWd[cols, :]),
           "trace": trace, "trace_grouped": trace_g, "backward_groups": bgroups, "err_dX_grouped": err(dXg, rdX[rows]),
           "err_dWg_grouped": err(gWg, rdWg[:, cols]), "err_dWu_grouped": err(gWu, rdWu[:, cols]),
           "err_dWd_grouped": err(gWd, rdWd[cols, :])}
    dist.barrier()
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump(out, f)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
