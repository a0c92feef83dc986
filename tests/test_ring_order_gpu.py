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


# ---------------------------------------------------------------------------------------------------------------
# The DIRECTION of the ring.  The rotation test above cannot tell (r - t) mod D from (r + t) mod D: both depend on
# r - k only.  What can: fp32 absorption.  The inputs below are built so that, for every rank r,
#   * the shard met first, k = r, contributes +B to every accumulator (B about 2^23 .. 2^24.5, every partial sum exact),
#   * the shard met second, k = r - 1 (Algorithm 2: receive from p - 1), contributes exactly -B,
#   * every other shard contributes less than half a unit in the last place of B.
# In ring order the accumulator goes B, 0, then collects the small contributions exactly.  In the reversed order
# (r, r+1, ..., r-1) the small contributions are added to B, vanish, and the result is 0.  The same matrix of scales
# does it for Y, for dX (probe columns) and, read column-wise, for the order (k + t) mod D in which shard k's weight
# gradient meets the ranks.  The oracle (fp64, no absorption) gives the small sum; so does the GPU iff its order is right.
# ---------------------------------------------------------------------------------------------------------------
def _direction_inputs(S_loc, H, F_d, D, seed=7):
    rng = np.random.Generator(np.random.Philox(seed))
    S, F = D * S_loc, D * F_d
    big, small = 2.0 ** 14, 2.0 ** -12
    h0 = D                                     # column of dY that is switched on
    X = np.zeros((S, H), np.float32)
    dY = np.zeros((S, H), np.float32)
    for r in range(D):
        X[r * S_loc:(r + 1) * S_loc, r] = 1.0  # rank r's tokens: the unit vector of feature r
    dY[:, h0] = 1.0
    W = rng.integers(1, 5, size=(F_d, H)).astype(np.float32)     # small integers: every product and sum is exact
    W2 = rng.integers(1, 5, size=(H, F_d)).astype(np.float32)
    Wg = np.tile(W2, (1, D))                   # [H, F]; rows >= D only matter for dX = dG Wg^T (the probe columns)
    Wg[:D, :] = 1.0                            # G = X_r Wg_k = 1 for every rank and shard
    Wu = np.zeros((H, F), np.float32)
    for r in range(D):
        for k in range(D):
            scale = big if k == r else (-big if k == (r - 1) % D else small)
            Wu[r, k * F_d:(k + 1) * F_d] = scale      # U_{r,k} = scale
    Wd = np.tile(W, (D, 1))                    # [F, H], the same block for every shard
    to_bits = inp.f32_to_bf16_bits
    host = inp.Inputs(to_bits(X), to_bits(Wg), to_bits(Wu), to_bits(Wd), to_bits(dY))
    for a, bts in ((X, host.X), (Wg, host.Wg), (Wu, host.Wu), (Wd, host.Wd), (dY, host.dY)):
        assert np.array_equal(inp.bf16_bits_to_f32(bts), a)      # everything is exactly representable in bf16
    return host, h0


def _sum_in_order(parts, order):
    """fp32 running sum of per-shard (or per-rank) contributions in the given order."""
    acc = np.zeros_like(parts[0], dtype=np.float32)
    for i in order:
        acc = (acc + parts[i].astype(np.float32)).astype(np.float32)
    return acc.astype(np.float64)


@pytest.mark.parametrize("S_loc,H,F_d,D", [(256, 256, 256, 5), (128, 256, 256, 3), (512, 512, 256, 4)])
def test_ring_direction_is_receive_from_the_left_neighbour(S_loc, H, F_d, D):
    from oracle import tsp_mlp_oracle as orc
    from tests.helpers import rel_fro, tensor_to_f64

    host, h0 = _direction_inputs(S_loc, H, F_d, D)
    S, F = D * S_loc, D * F_d
    prob = DeviceProblem(S, H, F, D, host=host, with_dy=True)
    X, Wg, Wu, Wd, dY = prob.f64()
    Y_ref = orc.gated_mlp_forward(X, Wg, Wu, Wd)
    rdX, rdWg, rdWu, rdWd = orc.gated_mlp_backward(X, Wg, Wu, Wd, dY)
    probe = np.arange(D + 1, H)                # columns of dX that only the dG Wg^T term reaches

    # --- the construction does what it claims: an fp32 sum in ring order keeps the small terms, the reversed one loses them
    for r in (0, D - 1):
        rows = slice(r * S_loc, r * S_loc + 4)
        parts = [orc.gated_mlp_forward(X[rows], Wg[:, k * F_d:(k + 1) * F_d], Wu[:, k * F_d:(k + 1) * F_d],
                                       Wd[k * F_d:(k + 1) * F_d]) for k in range(D)]
        ring_order = [(r - t) % D for t in range(D)]
        reversed_order = [(r + t) % D for t in range(D)]
        assert rel_fro(_sum_in_order(parts, ring_order), Y_ref[rows]) <= 1e-3
        assert rel_fro(_sum_in_order(parts, reversed_order), Y_ref[rows]) >= 0.9
    assert np.all(np.abs(Y_ref) > 0.05) and np.all(np.abs(Y_ref) < 10)

    # --- forward: Y in ring order
    got = tensor_to_f64(prob.forward())
    assert rel_fro(got, Y_ref) <= 1e-2, rel_fro(got, Y_ref)

    # --- backward: dX (probe columns) in ring order, dWd in the order shard k meets the ranks
    dX, dWg, dWu, dWd = prob.backward()
    gx = tensor_to_f64(dX)
    assert np.all(np.abs(rdX[:, probe]) > 0.1)
    assert rel_fro(gx[:, probe], rdX[:, probe]) <= 1e-2, rel_fro(gx[:, probe], rdX[:, probe])
    # (columns 0 .. D of dX also receive dU Wu^T, whose large terms cancel between shards that are not always met one
    # after the other: they are not part of this construction and are left out)
    gwd = inp.unshard_rows(tensor_to_f64(dWd))
    assert np.all(np.abs(rdWd[:, h0]) > 0.01)
    assert rel_fro(gwd[:, h0], rdWd[:, h0]) <= 1e-2, rel_fro(gwd[:, h0], rdWd[:, h0])
    assert rel_fro(gwd, rdWd) <= 1e-2
    assert rel_fro(inp.unshard_columns(tensor_to_f64(dWg)), rdWg) <= 1e-2
    assert rel_fro(inp.unshard_columns(tensor_to_f64(dWu)), rdWu) <= 1e-2
