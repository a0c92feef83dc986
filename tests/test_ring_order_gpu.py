"""The shard-visiting order is the ring's: rank r meets shard (r - t) mod D at step t, and shard k meets rank
(k + t) mod D.  That order depends only on the DIFFERENCE between rank and shard index, so renumbering ranks and shards
by the same rotation must reproduce every output bit for bit (rotated).  An order that treated shard 0 specially (all
ranks walking 0..D-1, say) would change each rank's fp32 accumulation order under the rotation, and with it some bits."""
import numpy as np
import pytest

from paper_2604_26294_b200 import build
from paper_2604_26294_b200 import inputs as inp
from tests.helpers import DeviceProblem

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build_library()


def _rotate_host(host, D):
    """Rank r gets rank (r-1)'s tokens, shard k gets shard (k-1)'s weights."""
    S, F = host.X.shape[0], host.Wd.shape[0]
    s_loc, f_d = S // D, F // D
    X = np.roll(host.X.reshape(D, s_loc, -1), 1, axis=0).reshape(S, -1)
    dY = np.roll(host.dY.reshape(D, s_loc, -1), 1, axis=0).reshape(S, -1)
    Wg = np.roll(host.Wg.reshape(-1, D, f_d), 1, axis=1).reshape(-1, F)
    Wu = np.roll(host.Wu.reshape(-1, D, f_d), 1, axis=1).reshape(-1, F)
    Wd = np.roll(host.Wd.reshape(D, f_d, -1), 1, axis=0).reshape(F, -1)
    return inp.Inputs(np.ascontiguousarray(X), np.ascontiguousarray(Wg), np.ascontiguousarray(Wu),
                      np.ascontiguousarray(Wd), np.ascontiguousarray(dY))


@pytest.mark.parametrize("S,H,F,D", [(512, 256, 512, 4), (2048, 512, 2048, 4), (3072, 256, 1536, 3)])
def test_outputs_are_invariant_under_a_joint_rotation_of_ranks_and_shards(S, H, F, D):
    import torch

    host = inp.make_inputs(S, H, F, seed=61, with_dy=True)
    a = DeviceProblem(S, H, F, D, host=host, with_dy=True)
    b_ = DeviceProblem(S, H, F, D, host=_rotate_host(host, D), with_dy=True)
    Ya, Yb = a.forward().clone(), b_.forward().clone()
    s_loc = S // D
    assert bool((torch.roll(Ya.view(D, s_loc, H), 1, 0).view(torch.int16) == Yb.view(D, s_loc, H).view(torch.int16)).all())
    dXa, dWga, dWua, dWda = a.backward()
    dXb, dWgb, dWub, dWdb = b_.backward()
    assert bool((torch.roll(dXa.view(D, s_loc, H), 1, 0).view(torch.int16) == dXb.view(D, s_loc, H).view(torch.int16)).all())
    for x, y in ((dWga, dWgb), (dWua, dWub), (dWda, dWdb)):
        assert bool((torch.roll(x, 1, 0).view(torch.int32) == y.view(torch.int32)).all())
