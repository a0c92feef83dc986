"""The multi-rank ring schedules (forward and backward with travelling gradient accumulators) over gloo on CPU."""
import json
import os

import pytest

from paper_2604_26294_b200 import ring
from tests.test_multi_rank_cpu import ROOT, _torchrun


def test_neighbours_and_shard_index():
    assert ring.ring_neighbours(0, 4) == (1, 3) and ring.ring_neighbours(3, 4) == (0, 2)
    for D in (1, 2, 3, 8):
        for r in range(D):
            met = [ring.shard_at_step(r, t, D) for t in range(D)]
            assert met[0] == r and sorted(met) == list(range(D))        # own shard first, every shard once
            assert all(ring.shard_at_step((r + 1) % D, t + 1, D) == met[t] for t in range(D - 1))  # it moves to p+1


@pytest.mark.parametrize("world", [2, 3, 4, 5])   # 3 and 4: p+1 and p-1 are different ranks, a reversed ring would show
def test_ring_schedules_reach_the_unsharded_result(tmp_path, world):
    res = _torchrun([os.path.join(ROOT, "tests", "ring_worker.py"), str(tmp_path)], nproc=world)
    assert res.returncode == 0, res.stderr[-3000:]
    for r in range(world):
        o = json.load(open(tmp_path / f"rank{r}.json"))
        assert o["visited"] == [(r - t) % world for t in range(world)]
        assert o["hook_calls"] == list(range(world - 1))      # once before every transfer, none after the last step
        assert [g[:2] for g in o["groups"]] == [[t0, min(2, world - t0)] for t0 in range(0, world, 2)]
        assert [g[2] for g in o["groups"]] == [t0 % 4 for t0 in range(0, world, 2)]
        for key in ("err_Y", "err_Y_grouped", "err_dX", "err_dWg", "err_dWu", "err_dWd", "err_dX_grouped",
                    "err_dWg_grouped", "err_dWu_grouped", "err_dWd_grouped"):
            assert o[key] <= 1e-12, (r, key, o[key])
        # the accumulator of shard r (this rank's own) was added to by the ranks r, r+1, ..., r+D-1 (mod D), in that
        # order: the order in which the shard meets the ranks, with and without grouping
        want = 0
        for t in range(world):
            want = want * world + (r + t) % world
        assert o["trace"] == want and o["trace_grouped"] == want, (r, o["trace"], o["trace_grouped"], want)
        assert [g[:2] for g in o["backward_groups"]] == [[t0, min(2, world - t0)] for t0 in range(0, world, 2)]
